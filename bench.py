"""Benchmark of the DB-SpMSpV hot path on B200.

Workload at N=1: R-MAT scale 20, edge factor 16, fp32 values, with the
input-sparsity sweep x nnz fraction 1e-5 ... 0.5.  One *step* is one pass of the whole hot path
(vector blocking -> selector -> worklist -> block microkernels -> writeback -> compaction) over
that batch: one dbspmspv_run call per sweep point, six calls.  L2 is flushed before every timed
call, so every number is cold.  `value` is the bytes the method must touch (B_touch, defined at
ByteModel below) summed over the sweep, divided by the summed device time.  DB-BFS GTEPS on the
symmetrised R-MAT scale 22 graph is reported in `bfs` unless --no-bfs is given.

python bench.py [--gpus N --steps K --warmup W] [--impl reference] [--no-bfs]
Under torchrun every rank runs the same sweep on its own GPU (independent replicas: the path
has no exchange step), times are the max over ranks, `value` is the whole-job aggregate.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2608_16308_b200 import workloads as wl  # noqa: E402

METRIC = "spmspv_sweep_achieved_hbm_GBps"
UNIT = "GB/s"
WORKLOAD = "rmat20_ef16_fp32_xsweep_1e-5..0.5"
VIEW_ENTRY_BYTES = 9          # idx 4 + w 4 + aux 1 per view entry


# ---------------------------------------------------------------------------------------------
# Algorithmic bytes (host, from the structure of A and x)
# ---------------------------------------------------------------------------------------------
def payload_bytes_per_entry(cls: np.ndarray, nnz: np.ndarray, vsize: int) -> np.ndarray:
    """Payload bytes of every view entry from the documented per-class sizes."""
    out = np.zeros(cls.size, dtype=np.int64)
    coo = cls == 1
    out[coo] = ((nnz[coo] + 3) // 4) * 4 + nnz[coo] * vsize
    mid = (cls >= 2) & (cls <= 4)
    out[mid] = (48 + nnz[mid] * vsize) if vsize else 32
    out[cls == 5] = 32 + 256 * vsize
    return ((out + 15) // 16) * 16          # every block is padded to 16 bytes


class ByteModel:
    """Algorithmic bytes of one SpMSpV call, each distinct byte once.
    B_touch: what the method must touch -- the view entries (9 bytes each) and payloads of the
    blocks in active column blocks, a column-pointer pair per active column block, x (8 bytes per
    listed nonzero, plus mask and staged block per nonempty vector block), y (8 bytes out and an
    8-byte accumulator read-modify-write per output, 8 bytes of hit flags per touched row block).
    B_min: the information-theoretic floor of a plain CSC gather -- per listed x_j its column's
    entries at (value + 4-byte row) each plus a pointer pair, x and y once."""

    def __init__(self, csr: wl.CSR, entry_col: np.ndarray, entry_cls: np.ndarray, entry_nnz: np.ndarray,
                 vsize: int):
        self.csr, self.vsize = csr, vsize
        nb = (csr.n + 15) // 16
        per_entry = VIEW_ENTRY_BYTES + payload_bytes_per_entry(entry_cls, entry_nnz, vsize)
        self.colblock_bytes = np.bincount(entry_col, weights=per_entry, minlength=nb)
        self.col_nnz = np.bincount(csr.col_idx, minlength=csr.n)

    def bytes(self, x_idx: np.ndarray, y_nnz: int, y_row_blocks: int):
        xb = np.unique(x_idx >> 4)
        touched = float(self.colblock_bytes[xb].sum())               # view entries + payload
        pointers = 8.0 * xb.size                                      # column-pointer pair
        xbytes = 8.0 * x_idx.size + xb.size * (2 + 64)                # list + mask + staged block
        ybytes = 8.0 * y_nnz + 8.0 * y_nnz + 8.0 * y_row_blocks       # out + acc RMW + mask set/clear
        b_touch = touched + pointers + xbytes + ybytes
        b_min = float((8 + self.col_nnz[x_idx] * (self.vsize + 4)).sum()) + 8.0 * x_idx.size + 8.0 * y_nnz
        return b_touch, b_min, touched + pointers + xb.size * 66     # last: traversal kernel only


# ---------------------------------------------------------------------------------------------
def sample_clocks(stop: threading.Event, out: list) -> None:
    q = "clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown," \
        "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap"
    idx = os.environ.get("LOCAL_RANK", "0")
    while not stop.is_set():
        try:
            r = subprocess.run(["nvidia-smi", f"--query-gpu={q}", "--format=csv,noheader,nounits", "-i", idx],
                               capture_output=True, text=True, timeout=5)
            if r.returncode == 0 and r.stdout.strip():
                out.append([f.strip() for f in r.stdout.strip().split(",")])
        except Exception:
            pass
        stop.wait(0.2)


def clocks_summary(samples: list) -> dict:
    if not samples:
        return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
    sm = sorted(int(s[0]) for s in samples if s[0].isdigit())
    names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
    reasons = [n for k, n in enumerate(names) if any(len(s) > 2 + k and s[2 + k].lower().startswith("active") for s in samples)]
    return {"sm_mhz": sm[len(sm) // 2] if sm else None,
            "sm_max_mhz": int(samples[0][1]) if samples[0][1].isdigit() else None,
            "reasons": reasons, "samples": len(samples)}


def max_over_ranks(value: float, device=None) -> float:
    """Max of a per-rank time over all ranks (the whole job is as slow as its slowest rank);
    identity without a process group.  Works on NCCL (device tensor) and gloo (CPU tensor)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank: float, ms_per_step_local: float, world: int, device=None):
    """Whole-job throughput of independent replicas: every rank processes `units_per_rank`
    per step, the step takes the max over ranks.  Returns (units per second, ms)."""
    ms = max_over_ranks(ms_per_step_local, device)
    return world * units_per_rank / (ms * 1e-3), ms


def measured_peak_gbs():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


# ---------------------------------------------------------------------------------------------
def reference_arm(args) -> None:
    """--impl reference: the CPU oracle as it stands, on the host cores, same config and metric."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    a = wl.rmat(20, 16, seed=1)
    A = oracle.RefMatrix(a.m, a.n, a.row_ptr, a.col_idx, a.val)
    A.csc()
    xs = [wl.rmat_x(a.n, f, k) for k, f in enumerate(wl.RMAT_SWEEP)]
    model = host_byte_model(a)
    per_step = []
    btouch_step = 0.0
    for it in range(args.warmup + args.steps):
        t_step, btouch_step = 0.0, 0.0
        for x in xs:
            best = None
            for fn in (oracle.ref_push, oracle.ref_pull):
                t0 = time.perf_counter()
                yi, _, _ = fn(A, x.idx, x.val)
                dt = time.perf_counter() - t0
                best = dt if best is None or dt < best else best
            t_step += best
            btouch_step += model.bytes(x.idx, yi.size, np.unique(yi >> 4).size)[0]
        if it >= args.warmup:
            per_step.append(t_step)
    ms = 1e3 * float(np.mean(per_step))
    value = btouch_step / (ms * 1e-3) / 1e9
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "note": "CPU oracle (Algorithm 1 push/pull, faster of the two per point), "
                                                     "whole sweep per step, single thread"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle",
                             "sample": "whole 6-point sweep per step"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def host_byte_model(a: wl.CSR) -> ByteModel:
    """Byte model with the class census computed on the host (used by the reference arm, where
    no GPU library is loaded): the documented classification rule applied with numpy."""
    rows = a.rows()
    key = (rows.astype(np.int64) >> 4) * ((a.n + 15) // 16) + (a.col_idx >> 4)
    ub, cnt = np.unique(key, return_counts=True)
    bcol = (ub % ((a.n + 15) // 16)).astype(np.int64)
    # blocks with fewer than 32 entries are INLINE (one 9-byte view entry per element, the
    # library's default); the handful of denser blocks are counted as CSR-class or Dense
    inl = cnt < 32
    cls = np.where(inl, 0, np.where(cnt < 32, 1, np.where(cnt > 128, 5, 4))).astype(np.int32)
    ecol = np.concatenate([np.repeat(bcol[inl], cnt[inl]), bcol[~inl]])
    ecls = np.concatenate([np.zeros(int(cnt[inl].sum()), np.int32), cls[~inl]])
    ennz = np.concatenate([np.ones(int(cnt[inl].sum()), np.int64), cnt[~inl]])
    return ByteModel(a, ecol, ecls, ennz, 4)


# ---------------------------------------------------------------------------------------------
def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-bfs", action="store_true")
    ap.add_argument("--bfs-scale", type=int, default=22)
    ap.add_argument("--bfs-only", action="store_true",
                    help="run only the DB-BFS leg and print its record (the command ncu captures k_bfs from)")
    ap.add_argument("--decode-only", action="store_true",
                    help="run only the decode layers and print their records (the command ncu captures k_decode_fused from)")
    ap.add_argument("--crossover", action="store_true",
                    help="print the measured push/pull crossover table (forced paths) and exit")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        reference_arm(args)
        return
    if args.crossover:
        crossover_table()
        return

    import torch
    import torch.distributed as dist
    from paper_2608_16308_b200 import binding as B

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    if args.bfs_only:
        if rank == 0:
            flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
            print(json.dumps(bench_bfs(args, B, torch, dev, flush)))
        return
    if args.decode_only:
        if rank == 0:
            flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
            print(json.dumps(decode_layers(B, torch, dev, cold_call_timer(torch, flush))))
        return
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    up = lambda arr: torch.from_numpy(np.ascontiguousarray(arr)).to(dev)
    a = wl.rmat(20, 16, seed=1)
    h = B.dbspmspv_create_csr(a.m, a.n, a.nnz, up(a.row_ptr), up(a.col_idx), up(a.val), B.F32)
    st0 = B.dbspmspv_get_stats(h)
    ne = int(st0.n_view_entries)
    e_col = torch.empty(ne, dtype=torch.int32, device=dev)
    e_cls = torch.empty(ne, dtype=torch.int32, device=dev)
    e_nnz = torch.empty(ne, dtype=torch.int32, device=dev)
    B.dbspmspv_export_blocks(h, None, e_col, e_cls, e_nnz)
    model = ByteModel(a, e_col.cpu().numpy().astype(np.int64), e_cls.cpu().numpy(), e_nnz.cpu().numpy().astype(np.int64), 4)
    del e_col, e_cls, e_nnz

    xs = [wl.rmat_x(a.n, f, k) for k, f in enumerate(wl.RMAT_SWEEP)]
    xd = [(up(x.idx), up(x.val)) for x in xs]
    xh = [(torch.from_numpy(x.idx).pin_memory(), torch.from_numpy(x.val).pin_memory()) for x in xs]
    y_idx = torch.empty(a.m, dtype=torch.int32, device=dev)
    y_val = torch.empty(a.m, dtype=torch.float32, device=dev)
    y_nnz = torch.zeros(1, dtype=torch.int32, device=dev)
    y_idx_h = torch.empty(a.m, dtype=torch.int32).pin_memory()
    y_val_h = torch.empty(a.m, dtype=torch.float32).pin_memory()
    y_nnz_h = torch.zeros(1, dtype=torch.int32).pin_memory()
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)     # > 126 MB L2
    stream = torch.cuda.current_stream()
    opts = B.default_run_opts()

    npts = len(xs)
    ev = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(npts)]
          for _ in range(args.steps)]
    kernel_ms = np.zeros((args.steps, npts))
    info = [None] * npts

    def one_call(k):
        B.dbspmspv_run(h, xd[k][0], xd[k][1], int(xs[k].idx.size), B.PLUS_TIMES, y_idx, y_val, a.m, y_nnz)

    for _ in range(args.warmup):
        for k in range(npts):
            flush.fill_(1)
            one_call(k)
    torch.cuda.synchronize()
    # separate pass with the library's kernel timing on (two extra event records per call):
    # duration of the traversal kernel alone, and the per-point facts for the byte model
    opts.timing = 1
    B.dbspmspv_set_run_opts(h, opts)
    for s in range(args.steps):
        for k in range(npts):
            flush.fill_(s & 0xFF)
            one_call(k)
            stt = B.dbspmspv_get_stats(h)        # synchronises; reads the traversal-kernel time
            kernel_ms[s, k] = stt.last_compute_ms
            if info[k] is None:
                yk = int(stt.last_y_nnz)
                yrb = int(torch.unique(y_idx[:yk] >> 4).numel())
                info[k] = (stt.last_path, stt.last_n_nzblk, stt.last_n_tasks, yk, yrb)
    opts.timing = 0
    B.dbspmspv_set_run_opts(h, opts)
    torch.cuda.synchronize()
    launches0 = B.dbspmspv_get_stats(h).kernel_launches

    stop, samples = threading.Event(), []
    th = threading.Thread(target=sample_clocks, args=(stop, samples), daemon=True)
    th.start()
    barrier()
    t_wall0 = time.perf_counter()
    for s in range(args.steps):
        for k in range(npts):
            flush.fill_(s & 0xFF)                # L2 flush, outside the event pair
            ev[s][k][0].record(stream)
            one_call(k)
            ev[s][k][1].record(stream)
    barrier()
    t_wall = time.perf_counter() - t_wall0
    stop.set()
    th.join(timeout=2)
    launches = B.dbspmspv_get_stats(h).kernel_launches - launches0

    call_ms = np.array([[ev[s][k][0].elapsed_time(ev[s][k][1]) for k in range(npts)] for s in range(args.steps)])
    step_ms = call_ms.sum(axis=1)
    ms_per_step = max_over_ranks(float(step_ms.mean()), dev)

    # ---- end to end through the same C-ABI call with HOST buffers: x and y live in page-locked
    # host memory that the device addresses directly, so the call's own kernels read x and write
    # y (and the count) across PCIe -- no staging copy, one synchronisation per call
    e2e_ms = []
    h2d = d2h = 0
    for s in range(max(3, args.steps // 2) + 2):
        tot = 0.0
        h2d = d2h = 0
        for k in range(npts):
            flush.fill_(1)
            n_x = int(xs[k].idx.size)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            B.dbspmspv_run(h, xh[k][0], xh[k][1], n_x, B.PLUS_TIMES, y_idx_h, y_val_h, a.m, y_nnz_h)
            e1.record(stream)
            stream.synchronize()
            kk = int(y_nnz_h.item())
            tot += e0.elapsed_time(e1)
            # x is read once by the blocking kernel; its indices once more by the clean-up pass
            # unless the dense copy is cleared wholesale (x lists more than n / 8 columns)
            h2d += 8 * n_x + (0 if 8 * n_x > a.n else 4 * n_x)
            d2h += 4 + 8 * kk
        if s >= 2:
            e2e_ms.append(tot)
    e2e_ms_step = max_over_ranks(float(np.mean(e2e_ms)), dev)

    peak, peak_kind = measured_peak_gbs()
    sweep, b_touch_total = [], 0.0
    for k, x in enumerate(xs):
        path, nzblk, ntasks, yk, yrb = info[k]
        bt, bm, bk = model.bytes(x.idx, yk, yrb)
        us = float(np.median(call_ms[:, k])) * 1e3
        kus = float(np.median(kernel_ms[:, k])) * 1e3
        b_touch_total += bt
        sweep.append({"x_fraction": wl.RMAT_SWEEP[k], "x_nnz": int(x.idx.size), "path": "push" if path == B.PATH_PUSH else "pull",
                      "us": round(us, 2), "us_min": round(float(call_ms[:, k].min()) * 1e3, 2),
                      "traversal_kernel_us": round(kus, 2), "y_nnz": yk, "n_nzblk": nzblk,
                      "B_touch": int(bt), "B_min": int(bm), "GBps_touch": round(bt / us / 1e3, 2),
                      "frac_of_peak_touch": round(bt / us / 1e3 / peak, 4), "frac_of_peak_min": round(bm / us / 1e3 / peak, 4)})
    value = world * b_touch_total / (ms_per_step * 1e-3) / 1e9
    e2e_value = world * b_touch_total / (e2e_ms_step * 1e-3) / 1e9
    # roofline of the dominant kernel: the traversal kernel at the sweep point that moves the
    # most bytes (x = 50 %, pull); achieved = its algorithmic bytes / its own duration, measured
    # with CUDA events recorded inside the library around that launch
    kdom = int(np.argmax([model.bytes(x.idx, info[k][3], info[k][4])[2] for k, x in enumerate(xs)]))
    b_kernel_dom = model.bytes(xs[kdom].idx, info[kdom][3], info[kdom][4])[2]
    kernel_dom_ms = float(np.median(kernel_ms[:, kdom]))
    achieved = b_kernel_dom / (kernel_dom_ms * 1e-3) / 1e9
    line = {"metric": METRIC, "value": round(value, 3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": round(ms_per_step, 5), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": WORKLOAD, "step": "6 dbspmspv_run calls (one per sweep point), auto path",
                       "l2": "flushed (512 MB write) before every timed call", "block_size": 16,
                       "parallelism": f"replicas x{world}" if world > 1 else "single GPU"},
            "e2e": {"value": round(e2e_value, 3), "unit": UNIT, "ms_per_step": round(e2e_ms_step, 5),
                    "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h)},
            "gpu_launches": int(launches),
            "clocks": clocks_summary(samples),
            "roofline": {"bound": "hbm", "kernel": f"k_compute, x fraction {wl.RMAT_SWEEP[kdom]} ({sweep[kdom]['path']})",
                         "achieved": round(achieved, 2), "peak": peak, "peak_kind": f"of {peak_kind}",
                         "unit": "GB/s", "frac": round(achieved / peak, 4), "traffic": NCU_TRAFFIC_BYTES_PER_LAUNCH,
                         "algorithmic_bytes_per_launch": int(b_kernel_dom),
                         "kernel_us": round(kernel_dom_ms * 1e3, 2)},
            "sweep": sweep, "wall_s_timed_region": round(t_wall, 3)}

    if rank == 0 and world == 1:
        line["cusparse_spmv_reference"] = cusparse_reference(a, torch, dev, flush)
        line["cpu_baseline"] = cpu_baseline(a, xs, model)
    if rank == 0 and world == 1 and not args.no_bfs:
        try:
            line["other_configs"] = other_configs(B, torch, dev, flush, peak)
        except Exception as e:
            line["other_configs"] = {"error": repr(e)}
        try:
            # hand the harness's cached device memory back first: with torch's allocator holding
            # the earlier legs' blocks the 3 GB graph format measured 6 % slower (same kernels)
            torch.cuda.empty_cache()
            line["bfs"] = bench_bfs(args, B, torch, dev, flush)
        except Exception as e:  # the SpMSpV line must survive a BFS-side problem
            line["bfs"] = {"error": repr(e)}
    B.dbspmspv_destroy(h)
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# DRAM traffic of that launch (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu capture
# summarised in profiles/k_compute_pull_rmat20_x50pct.txt
NCU_TRAFFIC_BYTES_PER_LAUNCH = 156602880


def crossover_table() -> None:
    """Forced push vs forced pull, whole dbspmspv_run call, cold L2, median of 15: the data
    behind the default th3 (Section 3.3.1's selector, crossover re-measured on B200)."""
    import torch
    from paper_2608_16308_b200 import binding as B
    dev = "cuda:0"
    torch.cuda.set_device(0)
    up = lambda arr: torch.from_numpy(np.ascontiguousarray(arr)).to(dev)
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)

    def timed(h, x, m, path):
        o = B.default_run_opts()
        o.force_path = path
        B.dbspmspv_set_run_opts(h, o)
        xi, xv = up(x.idx), up(x.val)
        y_idx = torch.empty(m, dtype=torch.int32, device=dev)
        y_val = torch.empty(m, dtype=torch.float32, device=dev)
        y_nnz = torch.zeros(1, dtype=torch.int32, device=dev)
        ts = []
        for it in range(18):
            flush.fill_(it)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            B.dbspmspv_run(h, xi, xv, int(x.idx.size), B.PLUS_TIMES, y_idx, y_val, m, y_nnz)
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1) * 1e3)
        return float(np.median(ts[3:]))

    print("| matrix | x | s_b = N_nzblk/N_blk | push us | pull us | faster |")
    print("|---|---|---|---|---|---|")
    cases = []
    a = wl.uniform_rows()
    cases.append(("uniform 16384^2, 8/row", a, [("164 nnz", wl.sparse_x(0, 1, a.n, 164))] +
                  [(f"{f:g}", wl.sparse_x(40 + i, 0, a.n, int(a.n * f))) for i, f in enumerate((0.05, 0.2, 0.5, 1.0))]))
    a2 = wl.rmat(20, 16, seed=1)
    fr = list(wl.RMAT_SWEEP) + [0.03, 0.05, 0.2, 0.3, 0.7, 1.0]
    cases.append(("R-MAT scale 20", a2, [(f"{f:g}", wl.rmat_x(a2.n, f, k) if k < 6 else wl.sparse_x(200 + k, 0, a2.n, int(a2.n * f)))
                                         for k, f in enumerate(fr)]))
    a3 = wl.stencil27(160, seed=2)
    cases.append(("27-pt stencil 160^3, runs of 64", a3, [(f"{r * 64 / a3.n:.3g}", wl.clustered_x(a3.n, r))
                                                          for r in (64, 3200, 12800, 32000)]))
    for name, mat, xs in cases:
        h = B.dbspmspv_create_csr(mat.m, mat.n, mat.nnz, up(mat.row_ptr), up(mat.col_idx), up(mat.val), B.F32)
        nblk = (mat.n + 15) // 16
        for label, x in sorted(xs, key=lambda t: t[1].idx.size):
            sb = np.unique(x.idx >> 4).size / nblk
            tp, tl = timed(h, x, mat.m, B.PATH_PUSH), timed(h, x, mat.m, B.PATH_PULL)
            print(f"| {name} | {label} | {sb:.4f} | {tp:.1f} | {tl:.1f} | {'push' if tp < tl else 'pull'} |")
        B.dbspmspv_destroy(h)


def cold_call_timer(torch, flush):
    """us of one call: L2 flushed before every call, median of 12 after 3 warm-ups, CUDA events."""
    def timed(fn):
        ts = []
        for it in range(15):
            flush.fill_(it)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1) * 1e3)
        return float(np.median(ts[3:]))
    return timed


def other_configs(B, torch, dev, flush, peak):
    """The remaining workload shapes, one record each (whole call, cold L2, median of 12 after 3
    warm-ups): the uniform matrix with a 1 % x, the 27-point stencil with clustered x at 0.1 %
    and 5 %, and single-token decode on three pruned layer shapes next to a dense bf16 GEMV of
    the same shape on the same box."""
    up = lambda arr: torch.from_numpy(np.ascontiguousarray(arr)).to(dev)
    out = []

    timed = cold_call_timer(torch, flush)

    def spmspv_case(name, a, xs):
        h = B.dbspmspv_create_csr(a.m, a.n, a.nnz, up(a.row_ptr), up(a.col_idx), up(a.val), B.F32)
        ne = int(B.dbspmspv_get_stats(h).n_view_entries)
        e_col = torch.empty(ne, dtype=torch.int32, device=dev)
        e_cls = torch.empty(ne, dtype=torch.int32, device=dev)
        e_nnz = torch.empty(ne, dtype=torch.int32, device=dev)
        B.dbspmspv_export_blocks(h, None, e_col, e_cls, e_nnz)
        model = ByteModel(a, e_col.cpu().numpy().astype(np.int64), e_cls.cpu().numpy(), e_nnz.cpu().numpy().astype(np.int64), 4)
        y_idx = torch.empty(a.m, dtype=torch.int32, device=dev)
        y_val = torch.empty(a.m, dtype=torch.float32, device=dev)
        y_nnz = torch.zeros(1, dtype=torch.int32, device=dev)
        for label, x in xs:
            xi, xv = up(x.idx), up(x.val)
            us = timed(lambda: B.dbspmspv_run(h, xi, xv, int(x.idx.size), B.PLUS_TIMES, y_idx, y_val, a.m, y_nnz))
            st = B.dbspmspv_get_stats(h)
            k = int(y_nnz.item())
            yrb = int(np.unique(y_idx[:k].cpu().numpy() >> 4).size)
            bt = model.bytes(x.idx, k, yrb)[0]
            out.append({"workload": name, "x": label, "path": "push" if st.last_path == B.PATH_PUSH else "pull",
                        "us": round(us, 2), "y_nnz": k, "B_touch": int(bt), "GBps_touch": round(bt / us / 1e3, 2),
                        "frac_of_peak_touch": round(bt / us / 1e3 / peak, 4)})
        B.dbspmspv_destroy(h)

    a1 = wl.uniform_rows()
    spmspv_case("uniform16384_8perrow_fp32", a1, [("164 nnz (1 %)", wl.sparse_x(0, 1, a1.n, 164))])
    a3 = wl.stencil27(160, seed=2)
    spmspv_case("stencil27_160cubed_fp32", a3, [("0.1 % in runs of 64", wl.clustered_x(a3.n, 64)),
                                                 ("5 % in runs of 64", wl.clustered_x(a3.n, 3200))])
    del a3
    out += decode_layers(B, torch, dev, timed)
    return out


def decode_layers(B, torch, dev, timed):
    """Single-token decode on the three pruned layer shapes (bf16, 50 % magnitude-pruned) at
    70 % and 90 % activation zeros, whole call, next to a dense bf16 GEMV of the same shape."""
    up = lambda arr: torch.from_numpy(np.ascontiguousarray(arr)).to(dev)
    out = []
    for (m, n) in wl.DECODE_SHAPES:
        wgt = wl.pruned_weight(m, n, 0.5)
        bits = wl.f32_to_bf16_bits(wgt.val).view(np.int16)
        h = B.dbspmspv_create_csr(wgt.m, wgt.n, wgt.nnz, up(wgt.row_ptr), up(wgt.col_idx), up(bits), B.BF16)
        y = torch.empty(m, dtype=torch.float32, device=dev)
        wd = torch.randn(m, n, device=dev, dtype=torch.bfloat16)
        xb = torch.randn(n, device=dev, dtype=torch.bfloat16)
        gemv = timed(lambda: torch.mv(wd, xb))
        for zf in (0.7, 0.9):          # 0.9: the activation density of the paper's Table 2
            x = wl.relu_activation(n, zf)
            xd = up(wl.f32_to_bf16_bits(x).view(np.int16))
            us = timed(lambda: B.dbspmspv_decode(h, xd, y))
            st = B.dbspmspv_get_stats(h)
            out.append({"workload": f"decode_{m}x{n}_bf16_prune50_act{int(zf * 100)}zero", "path": "push" if st.last_path == B.PATH_PUSH else "pull",
                        "us": round(us, 2), "dense_bf16_gemv_us_same_box": round(gemv, 2),
                        "format_bytes": int(st.payload_bytes + st.csr_view_bytes)})
        B.dbspmspv_destroy(h)
        del wd
    return out


def cusparse_reference(a, torch, dev, flush):
    """Same-box library reference: CSR SpMV on x densified to length n (torch's sparse CSR
    matmul, which calls cuSPARSE).  One time serves every sweep point: a dense x makes the
    library read the whole matrix whatever x holds.  Harness only; the library never links it."""
    try:
        A = torch.sparse_csr_tensor(torch.from_numpy(a.row_ptr).to(dev), torch.from_numpy(a.col_idx.astype(np.int64)).to(dev),
                                    torch.from_numpy(a.val).to(dev), size=(a.m, a.n))
        xd = torch.zeros(a.n, 1, dtype=torch.float32, device=dev)
        xd[:: 7] = 1.0
        ts = []
        for it in range(13):
            flush.fill_(it)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            y = A @ xd
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1) * 1e3)
        return {"us": round(float(np.median(ts[3:])), 2), "what": "torch sparse CSR (cuSPARSE) SpMV, fp32, dense x, cold L2",
                "csr_bytes": int(a.nnz * 8 + (a.m + 1) * 8)}
    except Exception as e:
        return {"error": repr(e)}


def cpu_baseline(a, xs, model):
    """The oracle as it stands, single thread, on the same sweep (bounded: one pass, both
    routines per point, the faster one counted)."""
    import oracle
    A = oracle.RefMatrix(a.m, a.n, a.row_ptr, a.col_idx, a.val)
    A.csc()
    total_t, total_b = 0.0, 0.0
    for rep in range(2):
        total_t, total_b = 0.0, 0.0
        for x in xs:
            best = None
            for fn in (oracle.ref_push, oracle.ref_pull):
                t0 = time.perf_counter()
                yi, _, _ = fn(A, x.idx, x.val)
                dt = time.perf_counter() - t0
                best = dt if best is None or dt < best else best
            total_t += best
            total_b += model.bytes(x.idx, yi.size, np.unique(yi >> 4).size)[0]
    return {"value": round(total_b / total_t / 1e9, 4), "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": "whole 6-point sweep, faster of ref_push/ref_pull per point, second of two passes",
            "ms_per_step": round(total_t * 1e3, 3), "host_cores_available": os.cpu_count()}


def bench_bfs(args, B, torch, dev, flush):
    """DB-BFS GTEPS on the symmetrised R-MAT graph, 16 seeded sources (configs[3])."""
    g = wl.rmat(args.bfs_scale, 16, seed=3, values=False, symmetrise=True)
    up = lambda arr: torch.from_numpy(np.ascontiguousarray(arr)).to(dev)
    h = B.dbspmspv_create_csr(g.m, g.n, g.nnz, up(g.row_ptr), up(g.col_idx), None, B.PATTERN)
    srcs = wl.bfs_sources(g, 16)
    deg = np.diff(g.row_ptr)
    levels = torch.empty(g.n, dtype=torch.int32, device=dev)
    import oracle
    A = oracle.RefMatrix(g.m, g.n, g.row_ptr, g.col_idx)
    A.csc()
    times, teps, nlev, matches, cpu_s, cpu_edges = [], [], [], [], 0.0, 0.0
    for s in srcs:
        best = None
        for rep in range(3):
            flush.fill_(rep)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            B.db_bfs(h, int(s), levels)
            e1.record()
            torch.cuda.synchronize()
            t = e0.elapsed_time(e1)
            best = t if best is None or t < best else best
        lv = levels.cpu().numpy()
        edges = float(deg[lv >= 0].sum()) / 2.0
        times.append(best)
        teps.append(edges / (best * 1e-3) / 1e9)
        nlev.append(int(B.dbspmspv_get_stats(h).bfs_levels))
        t0 = time.perf_counter()
        ref = oracle.ref_bfs(A, int(s))               # every timed source is compared with the oracle
        cpu_s += time.perf_counter() - t0
        cpu_edges += float(deg[ref >= 0].sum()) / 2.0
        matches.append(bool(np.array_equal(ref, lv)))
    B.dbspmspv_destroy(h)
    hm = len(teps) / sum(1.0 / t for t in teps)
    return {"workload": f"rmat{args.bfs_scale}_sym_ef16_pattern_16sources", "gteps_harmonic_mean": round(hm, 3),
            "gteps_min": round(min(teps), 3), "gteps_max": round(max(teps), 3),
            "ms_median": round(float(np.median(times)), 4), "levels": nlev, "vertices": int(g.n), "nnz": int(g.nnz),
            "sources_matching_oracle": int(sum(matches)), "sources": len(matches),
            "cpu_baseline": {"value": round(cpu_edges / cpu_s / 1e9, 4), "unit": "GTEPS",
                             "cores": 1, "kind": "oracle", "sample": "queue BFS from each of the sources"}}


if __name__ == "__main__":
    main()
