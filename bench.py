"""Benchmark of the DB-SpMSpV hot path on B200.

Workload at N=1: R-MAT scale 20, edge factor 16, fp32 values, with the input-sparsity sweep
x nnz fraction 1e-5 ... 0.5.  One *step* is one pass of the whole hot path (vector blocking ->
selector -> worklist -> block microkernels -> writeback -> compaction) over that batch: one
dbspmspv_run call per sweep point, six calls.  L2 is flushed before every timed call, so the
headline numbers are cold; an L2-warm pass is reported beside them.

Bytes.  Three figures per call (ByteModel below, all computed on the host from the structure of
(A, x) and the format's documented sizes):
  B_moved  what the implementation reads and writes on the path it took, each distinct byte
           once (format bytes as the library's counting pass reports them, plus x and y);
           `value` = sum of B_moved over the sweep / summed device time;
  B_touch  the block-granular scope definition: every entry and payload of every column block
           under a nonempty vector block (what a purely block-granular method must touch);
  B_min    the format-independent floor of a plain CSC gather.

python bench.py [--gpus N --steps K --warmup W] [--impl reference] [--no-bfs] [--no-extras]
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
NOMINAL_HBM_GBS = 8000.0      # the nominal HBM3e figure, reported beside the measured copy bandwidth
LEAN_CHUNK = 256              # entries per chunk of the streaming pull (whole chunks are read)
PUSH, PULL = 1, 2


# ---------------------------------------------------------------------------------------------
# Algorithmic bytes (host, from the structure of A and x)
# ---------------------------------------------------------------------------------------------
def payload_bytes_of(nnz: np.ndarray, vsize: int, th0=32, th1=128) -> np.ndarray:
    """Payload bytes of a block with `nnz` stored elements under the default options: below th0
    none (its elements are INLINE view entries); up to th1 a mask-based block (48-byte header +
    values; pattern matrices: 32 bytes of masks); above, Dense (32 bytes of masks + 256 values);
    every block padded to 16 bytes."""
    out = np.where(nnz < th0, 0, np.where(nnz > th1, 32 + 256 * vsize, (48 + nnz * vsize) if vsize else 32))
    return ((out + 15) // 16) * 16


class ByteModel:
    """Byte counts of one SpMSpV call from the matrix structure alone (the library is not
    consulted: its counting pass, dbspmspv_count_call_bytes, is the cross-check)."""

    def __init__(self, csr: wl.CSR, vsize: int):
        self.csr, self.vsize = csr, vsize
        self.nb = (csr.n + 15) // 16
        rows = csr.rows()
        key = (rows.astype(np.int64) >> 4) * self.nb + (csr.col_idx >> 4)
        ub, inv, cnt = np.unique(key, return_inverse=True, return_counts=True)
        blk_col = (ub % self.nb).astype(np.int64)
        inline_blk = cnt < 32
        elem_inline = inline_blk[inv]
        pbytes = payload_bytes_of(cnt, vsize)
        self.col_nnz = np.bincount(csr.col_idx, minlength=csr.n)
        self.inline_col_nnz = np.bincount(csr.col_idx[elem_inline], minlength=csr.n)
        # per column block: entries with a payload, their payload bytes, all view entries
        pay = ~inline_blk
        self.cb_payload_entries = np.bincount(blk_col[pay], minlength=self.nb)
        self.cb_payload_bytes = np.bincount(blk_col[pay], weights=pbytes[pay], minlength=self.nb)
        self.cb_inline_entries = np.bincount(csr.col_idx[elem_inline] >> 4, minlength=self.nb)
        self.blk_col, self.blk_payload_bytes, self.blk_is_payload = blk_col, pbytes, pay
        self.n_inline = int(elem_inline.sum())
        self.n_payload = int(pay.sum())
        self.n_entries = self.n_inline + self.n_payload
        self.n_lean_rows = int(np.unique(rows[elem_inline]).size)
        self.heavy = 2 * int(cnt[pay].sum()) > csr.nnz        # most elements in blocks with a payload
        self.payload_total = float(pbytes.sum())

    # -- what the format part of a call reads (mirrors dbspmspv_count_call_bytes)
    def format_bytes(self, x_idx: np.ndarray, path: int) -> dict:
        xb = np.unique(x_idx >> 4)
        if path == PUSH:
            if self.heavy:
                entries = float((self.cb_payload_entries[xb] + self.cb_inline_entries[xb]).sum())
                pointers = 8.0 * xb.size
            else:
                entries = float(self.inline_col_nnz[x_idx].sum() + self.cb_payload_entries[xb].sum())
                pointers = 8.0 * x_idx.size + 8.0 * xb.size
            blocks = float(self.cb_payload_entries[xb].sum())
            payload = float(self.cb_payload_bytes[xb].sum())
        else:
            if x_idx.size == 0:
                return {"view_entries": 0, "view_bytes": 0, "payload_blocks": 0, "payload_bytes": 0, "pointer_bytes": 0,
                        "active_vector_blocks": 0}
            if self.heavy:
                raise NotImplementedError("pull tables of a payload-dominated handle come from the library's statistics")
            n_chunks = (self.n_entries + LEAN_CHUNK - 1) // LEAN_CHUNK
            entries = float(n_chunks * LEAN_CHUNK)
            pointers = 4.0 * (n_chunks + self.n_lean_rows + self.n_payload)
            active = np.zeros(self.nb, dtype=bool)
            active[xb] = True
            sel = self.blk_is_payload & active[self.blk_col]
            blocks = float(sel.sum())
            payload = float(self.blk_payload_bytes[sel].sum())
        return {"view_entries": int(entries), "view_bytes": int(VIEW_ENTRY_BYTES * entries), "payload_blocks": int(blocks),
                "payload_bytes": int(payload), "pointer_bytes": int(pointers), "active_vector_blocks": int(xb.size)}

    def moved(self, x_idx: np.ndarray, path: int, y_nnz: int, fmt: dict | None = None, one_kernel: bool = False) -> dict:
        """Bytes the implementation moves on `path`, each distinct byte once: the format part
        (above), x (the list, the dense copy written and gathered, the masks, the clean-up),
        y (accumulator read-modify-write, hit flags, the sorted output) and the two O(m) scans
        of the compaction passes (hit flags in, packed masks out and in).  one_kernel: the
        single-kernel form of a short call -- x is read once as a list, the row bitmap lives in
        shared memory (no scans), y is the accumulator read-modify-write, the row list written
        and read back, the gather-and-clear and the output."""
        f = fmt if fmt is not None else self.format_bytes(x_idx, path)
        m, nx = self.csr.m, x_idx.size
        if one_kernel:
            fmt_total = f["view_bytes"] + f["payload_bytes"] + f["pointer_bytes"]
            xbytes, ybytes = 8.0 * nx, 8.0 * y_nnz + 8.0 * y_nnz + 8.0 * y_nnz + 8.0 * y_nnz
            return {"format": fmt_total, "x": xbytes, "y": ybytes, "scans": 0.0, "total": fmt_total + xbytes + ybytes,
                    "traversal_kernel": fmt_total + xbytes + ybytes}
        xbytes = 8.0 * nx + 4.0 * nx + 4.0 * nx + 2.0 * f["active_vector_blocks"] + 4.0 * nx + 6.0 * nx
        if path == PULL:
            xbytes += self.csr.n / 8.0                       # the presence filter, read once per SM from L2
        ybytes = 8.0 * y_nnz + 2.0 * y_nnz + 8.0 * y_nnz + 8.0 * y_nnz
        scans = m * 1.0 + (m / 8.0) * 2.0
        fmt_total = f["view_bytes"] + f["payload_bytes"] + f["pointer_bytes"]
        return {"format": fmt_total, "x": xbytes, "y": ybytes, "scans": scans, "total": fmt_total + xbytes + ybytes + scans,
                "traversal_kernel": fmt_total + 4.0 * nx + 10.0 * y_nnz + (self.csr.n / 8.0 if path == PULL else 2.0 * f["active_vector_blocks"])}

    def touch(self, x_idx: np.ndarray, y_nnz: int, y_row_blocks: int) -> float:
        xb = np.unique(x_idx >> 4)
        entries = self.cb_payload_entries[xb] + self.cb_inline_entries[xb]
        touched = float((VIEW_ENTRY_BYTES * entries + self.cb_payload_bytes[xb]).sum())
        return touched + 8.0 * xb.size + 8.0 * x_idx.size + xb.size * 66 + 16.0 * y_nnz + 8.0 * y_row_blocks

    def floor(self, x_idx: np.ndarray, y_nnz: int) -> float:
        return float((8 + self.col_nnz[x_idx] * (self.vsize + 4)).sum()) + 8.0 * x_idx.size + 8.0 * y_nnz

    def storage(self) -> dict:
        """Stored bytes of the plain formats the blocked one replaces (32-bit indices)."""
        a = self.csr
        csr = a.nnz * (4 + self.vsize) + 4 * (a.m + 1)
        csc = a.nnz * (4 + self.vsize) + 4 * (a.n + 1)
        return {"csr_bytes": int(csr), "csr_plus_csc_bytes": int(csr + csc)}


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


def fractions(nbytes: float, us: float, peak: float) -> dict:
    gbs = nbytes / us / 1e3 if us > 0 else 0.0
    return {"GBps": round(gbs, 2), "frac_of_measured": round(gbs / peak, 4), "frac_of_nominal_8TBps": round(gbs / NOMINAL_HBM_GBS, 4)}


def ncu_traffic(name: str):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, parsed from
    the text summary of its ncu capture under profiles/ (None when there is none)."""
    scale = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}
    total, seen = 0.0, 0
    try:
        for line in open(os.path.join(ROOT, "profiles", name)):
            f = line.split()
            if len(f) == 3 and f[0] in ("dram__bytes_read.sum", "dram__bytes_write.sum") and f[1] in scale:
                total += float(f[2]) * scale[f[1]]
                seen += 1
    except OSError:
        return None
    return int(total) if seen == 2 else None


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
    model = ByteModel(a, 4)
    per_step = []
    bytes_step = 0.0
    for it in range(args.warmup + args.steps):
        t_step, bytes_step = 0.0, 0.0
        for x in xs:
            best = None
            for fn in (oracle.ref_push, oracle.ref_pull):
                t0 = time.perf_counter()
                yi, _, _ = fn(A, x.idx, x.val)
                dt = time.perf_counter() - t0
                best = dt if best is None or dt < best else best
            t_step += best
            # same numerator as the GPU arm: the bytes the library moves on its default path
            path = PUSH if np.float32(np.unique(x.idx >> 4).size) / np.float32(model.nb) < np.float32(0.9) else PULL
            bytes_step += model.moved(x.idx, path, yi.size, None, path == PUSH and x.idx.size <= 256)["total"]    # (short calls: the one-kernel form)
        if it >= args.warmup:
            per_step.append(t_step)
    ms = 1e3 * float(np.mean(per_step))
    value = bytes_step / (ms * 1e-3) / 1e9
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "note": "CPU oracle (Algorithm 1 push/pull, faster of the two per point), "
                                                     "whole sweep per step, single thread"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle",
                             "sample": "whole 6-point sweep per step"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------------
def stats_of(ts_us) -> dict:
    a = np.asarray(ts_us, dtype=np.float64)
    return {"us": round(float(np.median(a)), 2), "us_min": round(float(a.min()), 2), "us_p90": round(float(np.percentile(a, 90)), 2)}


def timed_calls(torch, fn, flush, reps: int, warm: bool = False):
    """Device time of `reps` calls of fn (CUDA events on the current stream); cold: L2 flushed
    (512 MB write) before every call, outside the event pair; warm: back to back, with a short
    spin kernel in front of the first event so that the host has enqueued the whole call before
    the device reaches it (otherwise a call of a few microseconds measures the host's launch
    rate, not the device)."""
    ts = []
    for it in range(reps + 3):
        if not warm:
            flush.fill_(it & 0xFF)
        else:
            torch.cuda._sleep(200000)          # ~0.1 ms of spinning; touches no memory
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        if it >= 3:
            ts.append(e0.elapsed_time(e1) * 1e3)
    return ts


def latency_floors(B, torch, dev, flush) -> dict:
    """Floors of the machine for the latency-bound calls: an empty kernel (launch + completion)
    and the time of one dependent load, through a random cycle larger than L2 (DRAM) and
    through one that fits in L2."""
    out = {}
    ts = timed_calls(torch, lambda: B.dbspmspv_probe_floor(0), flush, 30, warm=True)
    out["empty_kernel_us"] = round(float(np.median(ts)), 2)
    res = torch.zeros(1, dtype=torch.int32, device=dev)
    for label, n in (("dram", 64 << 20), ("l2", 1 << 20)):
        # one cycle through all n elements: i -> (i + stride) mod n with an odd stride is a
        # permutation with a single cycle when n is a power of two
        stride = (n // 2 + 12345) | 1
        chain = ((torch.arange(n, dtype=torch.int64, device=dev) + stride) % n).to(torch.int32)
        steps = 256
        ts = timed_calls(torch, lambda: B.dbspmspv_probe_floor(1, chain, 0, steps, res), flush, 10, warm=(label == "l2"))
        out[f"dependent_load_{label}_ns"] = round((float(np.median(ts)) - out["empty_kernel_us"]) * 1e3 / steps, 1)
        del chain
    return out


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-bfs", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the other configurations, the ablation and the storage table")
    ap.add_argument("--bfs-scale", type=int, default=22)
    ap.add_argument("--bfs-only", action="store_true",
                    help="run only the DB-BFS leg and print its record (the command ncu captures k_bfs from)")
    ap.add_argument("--decode-only", action="store_true",
                    help="run only the decode layers and print their records (the command ncu captures k_decode_fused from)")
    ap.add_argument("--stencil-only", action="store_true",
                    help="run only the 27-point stencil records (the command ncu captures the payload-staging push from)")
    ap.add_argument("--stencil-d", type=int, default=160, help="edge length of the stencil grid for --stencil-only")
    ap.add_argument("--crossover", action="store_true",
                    help="print the measured push/pull crossover table (forced paths) and exit")
    ap.add_argument("--ablation", action="store_true", help="print the block-format ablation and storage records and exit")
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
    peak, peak_kind = measured_peak_gbs()
    if args.bfs_only or args.decode_only or args.ablation or args.stencil_only:
        if rank == 0:
            flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
            if args.bfs_only:
                print(json.dumps(bench_bfs(args, B, torch, dev, flush, peak)))
            elif args.stencil_only:
                print(json.dumps(other_configs(B, torch, dev, flush, peak, None, args.stencil_d)))
            elif args.decode_only:
                print(json.dumps(decode_layers(B, torch, dev, flush, peak) + [decode_chain(B, torch, dev, flush)] + decode_batch(B, torch, dev, flush)))
            else:
                print(json.dumps({"format_ablation": format_ablation(B, torch, dev, flush), "storage": storage_table(B, torch, dev)}))
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
    model = ByteModel(a, 4)

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
    # which points run in the one-kernel form of a short call (one launch)
    one_kernel = []
    for k in range(npts):
        l0 = B.dbspmspv_get_stats(h).kernel_launches
        one_call(k)
        one_kernel.append(B.dbspmspv_get_stats(h).kernel_launches - l0 == 1)
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

    # L2-warm pass: the same calls back to back, no flush (small formats and vectors stay in L2;
    # never to be read as HBM bandwidth)
    warm_us = []
    for k in range(npts):
        warm_us.append(float(np.median(timed_calls(torch, lambda: one_call(k), flush, 10, warm=True))))

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

    sweep, b_moved_total, b_touch_total, b_min_total = [], 0.0, 0.0, 0.0
    moved_by_point = []
    for k, x in enumerate(xs):
        path, nzblk, ntasks, yk, yrb = info[k]
        counted = B.dbspmspv_count_call_bytes(h, xd[k][0], int(x.idx.size), path)
        fmt_model = model.format_bytes(x.idx, path)
        fmt_counted = {f: int(getattr(counted, f)) for f in fmt_model}
        mv = model.moved(x.idx, path, yk, fmt_model, one_kernel[k])
        moved_by_point.append(mv)
        bt, bm = model.touch(x.idx, yk, yrb), model.floor(x.idx, yk)
        st = stats_of(call_ms[:, k] * 1e3)
        kus = float(np.median(kernel_ms[:, k])) * 1e3
        b_moved_total += mv["total"]
        b_touch_total += bt
        b_min_total += bm
        rec = {"x_fraction": wl.RMAT_SWEEP[k], "x_nnz": int(x.idx.size), "path": "push" if path == B.PATH_PUSH else "pull"}
        rec.update(st)
        rec.update({"us_l2_warm": round(warm_us[k], 2), "traversal_kernel_us": round(kus, 2), "y_nnz": yk, "n_nzblk": nzblk,
                    "n_tasks": ntasks, "one_kernel_form": bool(one_kernel[k]), "B_moved": int(mv["total"]),
                    "B_moved_parts": {p: int(v) for p, v in mv.items() if p not in ("total", "traversal_kernel")},
                    "B_touch": int(bt), "B_min": int(bm),
                    "format_bytes_model_equals_counting_pass": fmt_model == fmt_counted,
                    "moved": fractions(mv["total"], st["us"], peak), "touch": fractions(bt, st["us"], peak),
                    "min": fractions(bm, st["us"], peak)})
        if not rec["format_bytes_model_equals_counting_pass"]:
            rec["format_bytes_model"], rec["format_bytes_counted"] = fmt_model, fmt_counted
        sweep.append(rec)
    value = world * b_moved_total / (ms_per_step * 1e-3) / 1e9
    e2e_value = world * b_moved_total / (e2e_ms_step * 1e-3) / 1e9
    # roofline of the dominant kernel: the traversal kernel at the sweep point that moves the
    # most bytes; achieved = its algorithmic bytes / its own duration, measured with CUDA events
    # recorded inside the library around that launch
    kdom = int(np.argmax([mv["traversal_kernel"] for mv in moved_by_point]))
    b_kernel_dom = moved_by_point[kdom]["traversal_kernel"]
    kernel_dom_ms = float(np.median(kernel_ms[:, kdom]))
    achieved = b_kernel_dom / (kernel_dom_ms * 1e-3) / 1e9
    dom_pull = info[kdom][0] == B.PATH_PULL
    dom_name = "k_pull_lean" if dom_pull else "k_compute"
    traffic = ncu_traffic("k_pull_lean_rmat20_x50pct.txt" if dom_pull else "k_compute_push_rmat20_x10pct.txt")
    line = {"metric": METRIC, "value": round(value, 3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": round(ms_per_step, 5), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": WORKLOAD, "step": "6 dbspmspv_run calls (one per sweep point), auto path",
                       "l2": "flushed (512 MB write) before every timed call", "block_size": 16,
                       "bytes": "B_moved: what the implementation reads and writes per call, each distinct byte once",
                       "parallelism": f"replicas x{world}" if world > 1 else "single GPU"},
            "value_on_B_touch": round(world * b_touch_total / (ms_per_step * 1e-3) / 1e9, 3),
            "value_on_B_min": round(world * b_min_total / (ms_per_step * 1e-3) / 1e9, 3),
            "e2e": {"value": round(e2e_value, 3), "unit": UNIT, "ms_per_step": round(e2e_ms_step, 5),
                    "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h)},
            "gpu_launches": int(launches),
            "clocks": clocks_summary(samples),
            "roofline": {"bound": "hbm", "kernel": f"{dom_name}, x fraction {wl.RMAT_SWEEP[kdom]} ({sweep[kdom]['path']})",
                         "achieved": round(achieved, 2), "peak": peak, "peak_kind": f"of {peak_kind}",
                         "unit": "GB/s", "frac": round(achieved / peak, 4), "frac_of_nominal_8TBps": round(achieved / NOMINAL_HBM_GBS, 4),
                         "traffic": traffic, "algorithmic_bytes_per_launch": int(b_kernel_dom),
                         "kernel_us": round(kernel_dom_ms * 1e3, 2)},
            "sweep": sweep, "wall_s_timed_region": round(t_wall, 3),
            "format": {"stored_bytes": int(st0.payload_bytes + st0.csr_view_bytes + st0.csc_view_bytes + st0.segment_bytes + st0.lean_index_bytes),
                       "bfs_index_bytes": int(st0.bfs_index_bytes), **model.storage()}}

    if rank == 0 and world == 1:
        line["latency_floors"] = latency_floors(B, torch, dev, flush)
        fl = line["latency_floors"]
        for rec in sweep:
            rec["us_over_empty_kernel"] = round(rec["us"] / max(fl["empty_kernel_us"], 1e-3), 1)
        line["cusparse_spmv_reference"] = cusparse_reference(a, torch, dev, flush)
        line["cpu_baseline"] = cpu_baseline(a, xs, model, info, one_kernel)
    if rank == 0 and world == 1 and not args.no_extras:
        try:
            line["other_configs"] = other_configs(B, torch, dev, flush, peak, line.get("latency_floors"))
        except Exception as e:
            line["other_configs"] = {"error": repr(e)}
        try:
            line["format_ablation"] = format_ablation(B, torch, dev, flush)
            line["storage"] = storage_table(B, torch, dev)
        except Exception as e:
            line["format_ablation"] = {"error": repr(e)}
    if rank == 0 and world == 1 and not args.no_bfs:
        try:
            # hand the harness's cached device memory back first: with torch's allocator holding
            # the earlier legs' blocks the 3 GB graph format measured 6 % slower (same kernels)
            B.dbspmspv_destroy(h)
            h = None
            torch.cuda.empty_cache()
            line["bfs"] = bench_bfs(args, B, torch, dev, flush, peak)
        except Exception as e:  # the SpMSpV line must survive a BFS-side problem
            line["bfs"] = {"error": repr(e)}
    if h is not None:
        B.dbspmspv_destroy(h)
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


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
        ts = timed_calls(torch, lambda: B.dbspmspv_run(h, xi, xv, int(x.idx.size), B.PLUS_TIMES, y_idx, y_val, m, y_nnz), flush, 15)
        return float(np.median(ts))

    print("| matrix | x | s_b = N_nzblk/N_blk | push us | pull us | faster |")
    print("|---|---|---|---|---|---|")
    cases = []
    a = wl.uniform_rows()
    cases.append(("uniform 16384^2, 8/row", a, [("164 nnz", wl.sparse_x(0, 1, a.n, 164))] +
                  [(f"{f:g}", wl.sparse_x(40 + i, 0, a.n, int(a.n * f))) for i, f in enumerate((0.05, 0.2, 0.5, 1.0))]))
    a2 = wl.rmat(20, 16, seed=1)
    fr = list(wl.RMAT_SWEEP) + [0.03, 0.05, 0.15, 0.2, 0.3, 0.7, 1.0]
    cases.append(("R-MAT scale 20", a2, [(f"{f:g}", wl.rmat_x(a2.n, f, k) if k < 6 else wl.sparse_x(200 + k, 0, a2.n, int(a2.n * f)))
                                         for k, f in enumerate(fr)]))
    a4 = banded_plus_random(1 << 19, 12, 6, seed=7)
    cases.append(("band of 12 + 6 random per row, n = 2^19", a4, [(f"{f:g}", wl.sparse_x(300 + i, 0, a4.n, int(a4.n * f)))
                                                                  for i, f in enumerate((0.001, 0.01, 0.05, 0.2, 0.5))]))
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


def banded_plus_random(n: int, band: int, extra: int, seed: int) -> wl.CSR:
    """A matrix between the hypersparse and the payload-dominated extremes: every row holds a
    band of `band` consecutive columns around the diagonal (dense-ish blocks) plus `extra`
    uniformly random columns (singleton blocks)."""
    rows = np.repeat(np.arange(n, dtype=np.int64), band + extra)
    off = np.tile(np.arange(band, dtype=np.int64) - band // 2, n).reshape(n, band)
    bandc = np.clip(np.arange(n, dtype=np.int64)[:, None] + off, 0, n - 1)
    rnd = (wl.rand_u64(seed, 0, np.arange(n * extra, dtype=np.uint64)) % np.uint64(n)).astype(np.int64).reshape(n, extra)
    cols = np.concatenate([bandc, rnd], axis=1).reshape(-1)
    key = np.unique(rows * n + cols)
    r, c = (key // n).astype(np.int64), (key % n).astype(np.int32)
    row_ptr = np.zeros(n + 1, dtype=np.int64)
    np.cumsum(np.bincount(r, minlength=n), out=row_ptr[1:])
    val = (wl.rand_f32(seed, 1, np.arange(key.size, dtype=np.uint64)) * 2.0 - 1.0).astype(np.float32)
    return wl.CSR(n, n, row_ptr, c, val)


def minplus_rows(B, torch, dev, flush, peak):
    """The (min, +) semiring: one product on the sweep's matrix at three x densities next to the
    (+, *) push on the same x, and db_sssp on the symmetrised weighted R-MAT scale 20 graph (four
    sources; one checked against the CPU Bellman-Ford oracle, which is timed on that source)."""
    import oracle
    up = lambda arr: torch.from_numpy(np.ascontiguousarray(arr)).to(dev)
    out = []
    a = wl.rmat(20, 16, seed=1)
    h = B.dbspmspv_create_csr(a.m, a.n, a.nnz, up(a.row_ptr), up(a.col_idx), up(a.val), B.F32)
    model = ByteModel(a, 4)
    y_idx = torch.empty(a.m, dtype=torch.int32, device=dev)
    y_val = torch.empty(a.m, dtype=torch.float32, device=dev)
    y_nnz = torch.zeros(1, dtype=torch.int32, device=dev)
    o = B.default_run_opts()
    o.force_path = B.PATH_PUSH
    B.dbspmspv_set_run_opts(h, o)
    for k, f in ((2, 1e-3), (3, 1e-2), (4, 1e-1)):
        x = wl.rmat_x(a.n, f, k)
        xi, xv = up(x.idx), up(x.val)
        rec = {"workload": "rmat20_ef16_fp32 (min,+) product", "x": f"x fraction {f:g}", "path": "push"}
        for name, sr in (("minplus", B.MIN_PLUS), ("plus_times_forced_push", B.PLUS_TIMES)):
            call = lambda: B.dbspmspv_run(h, xi, xv, int(x.idx.size), sr, y_idx, y_val, a.m, y_nnz)
            st = stats_of(timed_calls(torch, call, flush, 12))
            rec[name + "_us"] = st["us"]
            if sr == B.MIN_PLUS:
                kk = int(y_nnz.item())
                mv = model.moved(x.idx, B.PATH_PUSH, kk, None)
                rec.update({"y_nnz": kk, "B_moved": int(mv["total"]), "moved": fractions(mv["total"], st["us"], peak)})
        out.append(rec)
    B.dbspmspv_destroy(h)
    del a
    g = wl.rmat(20, 16, seed=3, symmetrise=True)
    g.val = (0.05 + wl.rand_f32(7, 1, np.arange(g.nnz))).astype(np.float32)
    h = B.dbspmspv_create_csr(g.m, g.n, g.nnz, up(g.row_ptr), up(g.col_idx), up(g.val), B.F32)
    dist = torch.empty(g.n, dtype=torch.float32, device=dev)
    srcs = wl.bfs_sources(g, 4)
    ms, steps, edges = [], [], []
    deg = np.diff(g.row_ptr)
    for s_ in srcs:
        B.db_sssp(h, int(s_), dist)                         # warm-up (the first call allocates)
        flush.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); n_steps = B.db_sssp(h, int(s_), dist); e1.record()
        torch.cuda.synchronize()
        dv = dist.cpu().numpy()
        ms.append(e0.elapsed_time(e1)); steps.append(n_steps); edges.append(int(deg[np.isfinite(dv)].sum()))
    t0 = time.perf_counter()
    want = oracle.ref_sssp(oracle.RefMatrix(g.m, g.n, g.row_ptr, g.col_idx, g.val), int(srcs[-1]))
    cpu_s = time.perf_counter() - t0
    fin = np.isfinite(want)
    ok = bool(np.array_equal(np.isfinite(dv), fin) and np.all(np.abs(dv[fin] - want[fin]) <= 64 * 2.0 ** -24 * want[fin] + 1e-30))
    out.append({"workload": "rmat20_ef16_symmetrised_weighted_fp32 db_sssp", "sources": len(srcs),
                "ms_per_search_median": round(float(np.median(ms)), 3), "ms_min": round(min(ms), 3), "ms_max": round(max(ms), 3),
                "products_per_search": steps, "edges_in_component": edges[-1],
                "GTEPS_edges_of_component_over_time": round(float(np.mean([e / (t * 1e-3) / 1e9 for e, t in zip(edges, ms)])), 3),
                "cpu_bellman_ford_s": round(cpu_s, 3), "matches_oracle": ok})
    if not ok:
        raise SystemExit("db_sssp disagrees with the oracle")
    B.dbspmspv_destroy(h)
    return out


def other_configs(B, torch, dev, flush, peak, floors, stencil_only_d=None):
    """The remaining workload shapes, one record each (whole call, cold L2 and L2-warm): the
    uniform matrix with a 1 % x, the 27-point stencil with clustered x at 0.1 % and 5 %, and
    single-token decode on three pruned layer shapes next to a dense bf16 GEMV of the same shape
    on the same box."""
    up = lambda arr: torch.from_numpy(np.ascontiguousarray(arr)).to(dev)
    out = []

    def spmspv_case(name, a, xs):
        h = B.dbspmspv_create_csr(a.m, a.n, a.nnz, up(a.row_ptr), up(a.col_idx), up(a.val), B.F32)
        model = ByteModel(a, 4)
        y_idx = torch.empty(a.m, dtype=torch.int32, device=dev)
        y_val = torch.empty(a.m, dtype=torch.float32, device=dev)
        y_nnz = torch.zeros(1, dtype=torch.int32, device=dev)
        for label, x in xs:
            xi, xv = up(x.idx), up(x.val)
            call = lambda: B.dbspmspv_run(h, xi, xv, int(x.idx.size), B.PLUS_TIMES, y_idx, y_val, a.m, y_nnz)
            st = stats_of(timed_calls(torch, call, flush, 12))
            warm = float(np.median(timed_calls(torch, call, flush, 10, warm=True)))
            stt = B.dbspmspv_get_stats(h)
            k = int(y_nnz.item())
            yrb = int(np.unique(y_idx[:k].cpu().numpy() >> 4).size)
            path = int(stt.last_path)
            counted = B.dbspmspv_count_call_bytes(h, xi, int(x.idx.size), path)
            fmt = {f: int(getattr(counted, f)) for f in ("view_entries", "view_bytes", "payload_blocks", "payload_bytes",
                                                          "pointer_bytes", "active_vector_blocks")}
            mv = model.moved(x.idx, path, k, fmt)       # format part from the counting pass (tables of a payload-dominated handle)
            bt, bm = model.touch(x.idx, k, yrb), model.floor(x.idx, k)
            rec = {"workload": name, "x": label, "path": "push" if path == B.PATH_PUSH else "pull"}
            rec.update(st)
            rec.update({"us_l2_warm": round(warm, 2), "y_nnz": k, "B_moved": int(mv["total"]), "B_touch": int(bt), "B_min": int(bm),
                        "moved": fractions(mv["total"], st["us"], peak), "touch": fractions(bt, st["us"], peak),
                        "min": fractions(bm, st["us"], peak)})
            if path == B.PATH_PUSH:
                rec["format_bytes_model_equals_counting_pass"] = model.format_bytes(x.idx, path) == fmt
            if floors:
                rec["us_over_empty_kernel"] = round(st["us"] / max(floors["empty_kernel_us"], 1e-3), 1)
            out.append(rec)
        B.dbspmspv_destroy(h)

    if stencil_only_d:          # (--stencil-only: the 27-point stencil alone, at a chosen edge length)
        a3 = wl.stencil27(stencil_only_d, seed=2)
        r1, r2 = max(1, round(1e-3 * a3.n / 64)), max(1, round(5e-2 * a3.n / 64))
        spmspv_case(f"stencil27_{stencil_only_d}cubed_fp32", a3, [("0.1 % in runs of 64", wl.clustered_x(a3.n, r1)),
                                                                   ("5 % in runs of 64", wl.clustered_x(a3.n, r2))])
        return out
    a1 = wl.uniform_rows()
    spmspv_case("uniform16384_8perrow_fp32", a1, [("164 nnz (1 %)", wl.sparse_x(0, 1, a1.n, 164))])
    a3 = wl.stencil27(160, seed=2)
    spmspv_case("stencil27_160cubed_fp32", a3, [("0.1 % in runs of 64", wl.clustered_x(a3.n, 64)),
                                                 ("5 % in runs of 64", wl.clustered_x(a3.n, 3200))])
    del a3
    # the sweep's matrix with its vertices relabelled by a seeded permutation (hubs scattered
    # instead of packed at the low indices): the 1 %, 10 % and 50 % points
    a2 = wl.rmat(20, 16, seed=1, relabel=True)
    spmspv_case("rmat20_ef16_relabelled_fp32", a2, [(f"x fraction {f:g}", wl.rmat_x(a2.n, f, k)) for k, f in ((3, 1e-2), (4, 1e-1), (5, 0.5))])
    del a2
    out += decode_layers(B, torch, dev, flush, peak)
    out.append(decode_chain(B, torch, dev, flush))
    out += decode_batch(B, torch, dev, flush)
    out += minplus_rows(B, torch, dev, flush, peak)
    return out


def decode_bytes(wgt: wl.CSR, x: np.ndarray) -> dict:
    """Bytes of one decode call on a pruned bf16 layer in its selective form: the whole block-CSR
    view (the pull walks it), under every nonempty vector block the block's 48-byte header
    (32-byte for Dense) and the 2-byte values of its active columns, x (2 bytes per entry) and
    y (4 per row).  (The streaming form moves the whole payload instead: see decode_layers.)
    B_min: the CSC floor -- per active column its entries at 2 + 4 bytes, x and y."""
    m, n = wgt.m, wgt.n
    rows = wgt.rows()
    nbk = (n + 15) // 16
    key = (rows.astype(np.int64) >> 4) * nbk + (wgt.col_idx >> 4)
    ub, inv, cnt = np.unique(key, return_inverse=True, return_counts=True)
    active_col = x != 0
    elem_active = active_col[wgt.col_idx]
    blk_active_vals = np.bincount(inv[elem_active], minlength=ub.size)
    cbmask = np.zeros(nbk, dtype=bool)
    cbmask[np.unique(np.flatnonzero(active_col) >> 4)] = True
    blk_touched = cbmask[(ub % nbk)]
    inline = cnt < 32
    n_entries = int(cnt[inline].sum() + (~inline).sum())
    header = np.where(cnt > 128, 32, 48)
    payload = float((header[blk_touched & ~inline]).sum() + 2.0 * blk_active_vals[blk_touched & ~inline].sum())
    moved = 9.0 * n_entries + 4.0 * ((m + 15) // 16 + 1) + payload + 2.0 * n + 4.0 * m
    col_nnz = np.bincount(wgt.col_idx, minlength=n)
    floor = float((8 + col_nnz[active_col] * 6).sum()) + 2.0 * n + 4.0 * m
    return {"B_moved_selective": int(moved), "B_min": int(floor), "payload_bytes_touched": int(payload), "view_entries": n_entries}


def decode_chain(B, torch, dev, flush):
    """A feed-forward pair chained on the device (Section 4.3 / 5.3): up projection 11008x4096,
    then down projection 4096x11008 whose x is the up projection's fp32 y with ReLU and a
    magnitude cut fused into the blocking (cut chosen for 10 % dense activations) -- two
    dbspmspv_decode calls, nothing in between.  Beside it: two dense bf16 GEMVs of the same
    shapes with torch's relu / cut / cast between them."""
    up = lambda arr: torch.from_numpy(np.ascontiguousarray(arr)).to(dev)
    n0, n1 = 4096, 11008
    hs = []
    for (m, n, stream) in ((n1, n0, 0), (n0, n1, 1)):
        wgt = wl.pruned_weight(m, n, 0.5, stream=stream)
        bits = wl.f32_to_bf16_bits(wgt.val).view(np.int16)
        hs.append(B.dbspmspv_create_csr(wgt.m, wgt.n, wgt.nnz, up(wgt.row_ptr), up(wgt.col_idx), up(bits), B.BF16))
        del wgt
    h_up, h_down = hs
    x0 = up(wl.f32_to_bf16_bits(wl.relu_activation(n0, 0.9)).view(np.int16))
    y1 = torch.empty(n1, dtype=torch.float32, device=dev)
    y2 = torch.empty(n0, dtype=torch.float32, device=dev)
    B.dbspmspv_decode(h_up, x0, y1)
    torch.cuda.synchronize()
    y1h = y1.cpu().numpy()
    tau = float(np.quantile(y1h, 0.9))                       # 10 % of the entries lie above it
    o = B.default_run_opts()
    o.decode_x_f32, o.decode_relu, o.decode_threshold = 1, 1, max(tau, 0.0)
    B.dbspmspv_set_run_opts(h_down, o)

    def chain():
        B.dbspmspv_decode(h_up, x0, y1)
        B.dbspmspv_decode(h_down, y1, y2)

    st = stats_of(timed_calls(torch, chain, flush, 12))
    warm = float(np.median(timed_calls(torch, chain, flush, 10, warm=True)))
    w1 = torch.randn(n1, n0, device=dev, dtype=torch.bfloat16)
    w2 = torch.randn(n0, n1, device=dev, dtype=torch.bfloat16)
    xb = torch.randn(n0, device=dev, dtype=torch.bfloat16)

    def dense():
        t = torch.mv(w1, xb)
        t = torch.where(t > tau, t, torch.zeros_like(t))
        return torch.mv(w2, t)

    gd = float(np.median(timed_calls(torch, dense, flush, 12)))
    density = float((wl.bf16_bits_to_f32(wl.f32_to_bf16_bits(y1h)) > max(tau, 0.0)).mean())
    for h in hs:
        B.dbspmspv_destroy(h)
    rec = {"workload": "decode_chain_up11008x4096_relu_cut_down4096x11008_bf16_prune50", "calls": 2,
           "x0_zero_fraction": 0.9, "x1_density_after_cut": round(density, 4), "us_l2_warm": round(warm, 2),
           "dense_bf16_gemv_pair_with_torch_relu_cut_us": round(gd, 2)}
    rec.update(st)
    return rec


def decode_batch(B, torch, dev, flush):
    """Multi-vector decode (the paper's stated limitation, Section 6): 2, 4 and 8 activation
    vectors through the 12288x4096 bf16 layer in one dbspmspv_decode_batch call (one pass over
    the payload, block products on the tensor cores), beside the same vectors as single calls
    and a dense bf16 GEMM of the same shape."""
    up = lambda arr: torch.from_numpy(np.ascontiguousarray(arr)).to(dev)
    m, n = wl.DECODE_SHAPES[0]
    wgt = wl.pruned_weight(m, n, 0.5)
    bits = wl.f32_to_bf16_bits(wgt.val).view(np.int16)
    h = B.dbspmspv_create_csr(wgt.m, wgt.n, wgt.nnz, up(wgt.row_ptr), up(wgt.col_idx), up(bits), B.BF16)
    wd = torch.randn(m, n, device=dev, dtype=torch.bfloat16)
    out = []
    for zf in (0.7, 0.9):
        xs = np.stack([wl.f32_to_bf16_bits(wl.relu_activation(n, zf, stream=50 + b)).view(np.int16) for b in range(8)])
        xd = up(xs)
        for batch in (2, 4, 8):
            y = torch.empty(batch, m, dtype=torch.float32, device=dev)
            call = lambda: B.dbspmspv_decode_batch(h, xd, n, y, m, batch)

            def singles():
                for b in range(batch):
                    B.dbspmspv_decode(h, xd[b], y[b])

            st = stats_of(timed_calls(torch, call, flush, 12))
            one = float(np.median(timed_calls(torch, singles, flush, 12)))
            xb = torch.randn(n, batch, device=dev, dtype=torch.bfloat16)
            gemm = float(np.median(timed_calls(torch, lambda: torch.mm(wd, xb), flush, 12)))
            rec = {"workload": f"decode_batch{batch}_{m}x{n}_bf16_prune50_act{int(zf * 100)}zero", "vectors": batch,
                   "single_calls_us": round(one, 2), "dense_bf16_gemm_us_same_box": round(gemm, 2)}
            rec.update(st)
            rec["us_per_vector"] = round(st["us"] / batch, 2)
            out.append(rec)
    B.dbspmspv_destroy(h)
    return out


def decode_layers(B, torch, dev, flush, peak):
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
        gemv = float(np.median(timed_calls(torch, lambda: torch.mv(wd, xb), flush, 12)))
        for zf in (0.7, 0.9):          # 0.9: the activation density of the paper's Table 2
            x = wl.relu_activation(n, zf)
            xd = up(wl.f32_to_bf16_bits(x).view(np.int16))
            call = lambda: B.dbspmspv_decode(h, xd, y)
            st = stats_of(timed_calls(torch, call, flush, 12))
            warm = float(np.median(timed_calls(torch, call, flush, 10, warm=True)))
            before = B.dbspmspv_get_stats(h).kernel_launches
            call()
            torch.cuda.synchronize()
            stt = B.dbspmspv_get_stats(h)
            streamed = stt.kernel_launches - before == 2       # zero kernel + streaming kernel; the selective form is one kernel
            db = decode_bytes(wgt, wl.bf16_bits_to_f32(wl.f32_to_bf16_bits(x)))
            # streaming form: the whole payload, the view entries with a payload (9 bytes), the
            # chunk table (16 bytes per chunk, part of segment_bytes), x once per thread block
            # (from L2 after the first: counted once), y zeroed and added to (4 + 8 bytes per row)
            db["B_moved"] = int(stt.payload_bytes + 9 * db["view_entries"] + stt.segment_bytes + 2 * n + 12 * m) if streamed else db["B_moved_selective"]
            rec = {"workload": f"decode_{m}x{n}_bf16_prune50_act{int(zf * 100)}zero", "path": "push" if stt.last_path == B.PATH_PUSH else "pull",
                   "form": "streaming" if streamed else "selective"}
            rec.update(st)
            rec.update({"us_l2_warm": round(warm, 2), "dense_bf16_gemv_us_same_box": round(gemv, 2),
                        "format_bytes": int(stt.payload_bytes + stt.csr_view_bytes), **db,
                        "moved": fractions(db["B_moved"], st["us"], peak), "min": fractions(db["B_min"], st["us"], peak)})
            out.append(rec)
        B.dbspmspv_destroy(h)
        del wd
    return out


def format_ablation(B, torch, dev, flush):
    """Block-format ablation (Section 5.4): COO-only / CSR-only / automatic block formats, forced
    pull, x density 0.1, whole call, cold L2 -- on a banded matrix with random fill-in and on the
    27-point stencil at 96^3."""
    up = lambda arr: torch.from_numpy(np.ascontiguousarray(arr)).to(dev)
    out = []
    mats = [("band12_plus_6random_n2^18", banded_plus_random(1 << 18, 12, 6, seed=7)), ("stencil27_96cubed", wl.stencil27(96, seed=2))]
    for name, a in mats:
        x = wl.sparse_x(77, 0, a.n, int(a.n * 0.1))
        y_idx = torch.empty(a.m, dtype=torch.int32, device=dev)
        y_val = torch.empty(a.m, dtype=torch.float32, device=dev)
        y_nnz = torch.zeros(1, dtype=torch.int32, device=dev)
        xi, xv = up(x.idx), up(x.val)
        rec = {"matrix": name, "nnz": int(a.nnz), "x_density": 0.1, "path": "pull (forced)"}
        for label, fmt in (("auto", B.FORMAT_AUTO), ("coo_only", B.FORMAT_COO), ("csr_only", B.FORMAT_CSR)):
            o = B.default_create_opts()
            o.force_format = fmt
            h = B.dbspmspv_create_csr(a.m, a.n, a.nnz, up(a.row_ptr), up(a.col_idx), up(a.val), B.F32, 16, o)
            ro = B.default_run_opts()
            ro.force_path = B.PATH_PULL
            B.dbspmspv_set_run_opts(h, ro)
            ts = timed_calls(torch, lambda: B.dbspmspv_run(h, xi, xv, int(x.idx.size), B.PLUS_TIMES, y_idx, y_val, a.m, y_nnz), flush, 8)
            us = float(np.median(ts))
            st = B.dbspmspv_get_stats(h)
            rec[label] = {"us": round(us, 1), "gflops_on_2nnz": round(2.0 * a.nnz / us / 1e3, 1),
                          "stored_bytes_per_nnz": round((st.payload_bytes + st.csr_view_bytes + st.csc_view_bytes) / a.nnz, 2)}
            B.dbspmspv_destroy(h)
        out.append(rec)
    return out


def modelled_block_size_bytes(a, vs: int, bs: int) -> dict:
    """Storage of the blocked format at block size `bs`, MODELLED on the host from the per-block
    element counts (the kernels exist for 16 x 16 blocks only; 32 and 64 are what the same layout
    rules would store): the class thresholds scale with the block area (no payload up to
    bs^2/8 - 1 elements, Dense above bs^2/2), a view entry is 8 bytes + the packed local
    coordinates, a mask-based block carries bs masks of bs bits and bs start offsets, a Dense
    block bs masks and bs^2 values; both views, their pointer arrays and the per-column
    pointers are counted.  At bs = 16 this is the library's own layout (checked against its
    statistics by the caller)."""
    rows = np.repeat(np.arange(a.m, dtype=np.int64), np.diff(a.row_ptr))
    nbc = (a.n + bs - 1) // bs
    key = (rows // bs) * nbc + (a.col_idx.astype(np.int64) // bs)
    cnt = np.unique(key, return_counts=True)[1]
    area = bs * bs
    th0, th1 = area // 8, area // 2
    coord = (2 * int(np.log2(bs)) + 7) // 8                 # bytes of a packed (row, column) pair
    start = 1 if area <= 256 else 2                         # bytes of a start offset
    inline = cnt < th0
    mid = (~inline) & (cnt <= th1)
    dense = cnt > th1
    r16 = lambda b: (b + 15) // 16 * 16
    payload = int(r16(bs * bs // 8 + bs * start + cnt[mid] * vs).sum()) if vs else int(r16(np.full(int(mid.sum()), bs * bs // 8)).sum())
    payload += int(dense.sum()) * int(r16(bs * bs // 8 + area * vs))
    entries = int(cnt[inline].sum()) + int(mid.sum()) + int(dense.sum())
    mb, nb = (a.m + bs - 1) // bs, nbc
    views = 2 * entries * (8 + coord) + 4 * (mb + 1) + 4 * (nb + 1) + 4 * (bs + 1) * nb
    return {"block": bs, "blocks": int(cnt.size), "no_payload_blocks": int(inline.sum()), "mask_blocks": int(mid.sum()),
            "dense_blocks": int(dense.sum()), "payload_bytes": payload, "view_bytes": int(views),
            "bytes_per_nnz": round((payload + views) / max(a.nnz, 1), 2)}


def storage_table(B, torch, dev):
    """Stored bytes of the blocked format against CSR and CSR + CSC (Section 5.5's accounting,
    on the synthetic inputs; 32-bit indices, the configuration's value type)."""
    up = lambda arr: None if arr is None else torch.from_numpy(np.ascontiguousarray(arr)).to(dev)
    out = []
    w = wl.pruned_weight(4096, 11008, 0.5)
    cases = [("uniform16384_8perrow_fp32", wl.uniform_rows(), B.F32, 4), ("rmat20_ef16_fp32", wl.rmat(20, 16, seed=1), B.F32, 4),
             ("stencil27_96cubed_fp32", wl.stencil27(96, seed=2), B.F32, 4), ("decode_4096x11008_bf16_prune50", w, B.BF16, 2),
             ("rmat18_sym_pattern", wl.rmat(18, 16, seed=3, values=False, symmetrise=True), B.PATTERN, 0)]
    for name, a, dt, vs in cases:
        val = None
        if dt == B.F32:
            val = a.val
        elif dt == B.BF16:
            val = wl.f32_to_bf16_bits(a.val).view(np.int16)
        h = B.dbspmspv_create_csr(a.m, a.n, a.nnz, up(a.row_ptr), up(a.col_idx), up(val), dt)
        st = B.dbspmspv_get_stats(h)
        fmt = int(st.payload_bytes + st.csr_view_bytes + st.csc_view_bytes + st.segment_bytes + st.lean_index_bytes)
        csr = a.nnz * (4 + vs) + 4 * (a.m + 1)
        both = 2 * a.nnz * (4 + vs) + 4 * (a.m + a.n + 2)
        sweep = [modelled_block_size_bytes(a, vs, bs) for bs in (16, 32, 64)]
        sweep[0]["payload_bytes_equals_library"] = sweep[0]["payload_bytes"] == int(st.payload_bytes)
        out.append({"matrix": name, "nnz": int(a.nnz), "format_bytes": fmt, "bfs_index_bytes": int(st.bfs_index_bytes),
                    "block_size_sweep_modelled": sweep,
                    "payload_bytes": int(st.payload_bytes), "view_bytes": int(st.csr_view_bytes + st.csc_view_bytes),
                    "csr_bytes": int(csr), "csr_plus_csc_bytes": int(both), "format_bytes_per_nnz": round(fmt / a.nnz, 2),
                    "vs_csr": round(fmt / csr, 3), "vs_csr_plus_csc": round(fmt / both, 3)})
        B.dbspmspv_destroy(h)
    return out


def cusparse_reference(a, torch, dev, flush):
    """Same-box library reference: CSR SpMV on x densified to length n (torch's sparse CSR
    matmul, which calls cuSPARSE), cold and L2-warm.  One time serves every sweep point: a dense
    x makes the library read the whole matrix whatever x holds.  Harness only; the library never
    links it."""
    try:
        A = torch.sparse_csr_tensor(torch.from_numpy(a.row_ptr).to(dev), torch.from_numpy(a.col_idx.astype(np.int64)).to(dev),
                                    torch.from_numpy(a.val).to(dev), size=(a.m, a.n))
        xd = torch.zeros(a.n, 1, dtype=torch.float32, device=dev)
        xd[:: 7] = 1.0
        cold = timed_calls(torch, lambda: A @ xd, flush, 10)
        warm = timed_calls(torch, lambda: A @ xd, flush, 10, warm=True)
        return {"us": round(float(np.median(cold)), 2), "us_l2_warm": round(float(np.median(warm)), 2),
                "what": "torch sparse CSR (cuSPARSE) SpMV, fp32, dense x", "csr_bytes": int(a.nnz * 8 + (a.m + 1) * 8)}
    except Exception as e:
        return {"error": repr(e)}


def cpu_baseline(a, xs, model, info, one_kernel):
    """The oracle as it stands, single thread, on the same sweep (bounded: one pass, both
    routines per point, the faster one counted; same byte numerator as the GPU line)."""
    import oracle
    A = oracle.RefMatrix(a.m, a.n, a.row_ptr, a.col_idx, a.val)
    A.csc()
    total_t, total_b = 0.0, 0.0
    for rep in range(2):
        total_t, total_b = 0.0, 0.0
        for k, x in enumerate(xs):
            best = None
            for fn in (oracle.ref_push, oracle.ref_pull):
                t0 = time.perf_counter()
                yi, _, _ = fn(A, x.idx, x.val)
                dt = time.perf_counter() - t0
                best = dt if best is None or dt < best else best
            total_t += best
            total_b += model.moved(x.idx, info[k][0], yi.size, None, one_kernel[k])["total"]
    return {"value": round(total_b / total_t / 1e9, 4), "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": "whole 6-point sweep, faster of ref_push/ref_pull per point, second of two passes",
            "ms_per_step": round(total_t * 1e3, 3), "host_cores_available": os.cpu_count()}


def bfs_level_bytes(g: wl.CSR, lv: np.ndarray, paths):
    """Algorithmic bytes per level of one DB-BFS run, from the graph and the levels it produced
    (an untimed host pass).  Push level: per frontier vertex 8 bytes of column pointers, per
    frontier edge 5 bytes of view entry (index word + coordinate byte) and 2 bytes of visited
    mask, per 32 edges an 8-byte task record written and read.  Pull level over the row-run
    index: per mask word 12 bytes (visited, next, spare), per row still wanted 8 bytes of row
    pointers, per entry scanned -- a row stops at its first frontier neighbour; entries come in
    aligned groups of four -- 4 bytes plus 2 bytes of frontier mask.  Both: 4 bytes of level
    and 4 of frontier word per vertex found."""
    deg = np.diff(g.row_ptr)
    out = []
    n_words = (g.n + 31) // 32
    for L, path in enumerate(paths):
        frontier = lv == L
        found = int((lv == L + 1).sum())
        if path == PUSH:
            edges = float(deg[frontier].sum())
            nbytes = 8.0 * frontier.sum() + 7.0 * edges + 16.0 * (edges / 32.0) + 8.0 * found
            out.append({"level": L, "path": "push", "frontier": int(frontier.sum()), "edges_walked": int(edges), "bytes": int(nbytes)})
        else:
            want = ((lv > L) | (lv < 0)) & (deg > 0)
            hit = frontier[g.col_idx]                              # entries whose column is in the frontier
            pos = np.flatnonzero(hit)
            row_of = np.searchsorted(g.row_ptr, pos, side="right") - 1
            first = np.full(g.n, -1, dtype=np.int64)
            keep = np.r_[True, row_of[1:] != row_of[:-1]] if pos.size else np.zeros(0, bool)
            first[row_of[keep]] = pos[keep]
            start, end = g.row_ptr[:-1], g.row_ptr[1:]
            stop = np.where(first >= 0, first + 1, end)            # scanned up to the first hit, else the whole row
            scanned = ((stop + 3) // 4) * 4 - (start // 4) * 4
            scanned = np.minimum(scanned, ((end + 3) // 4) * 4 - (start // 4) * 4)
            entries = float(scanned[want].sum())
            nbytes = 12.0 * n_words + 8.0 * want.sum() + 6.0 * entries + 8.0 * found
            out.append({"level": L, "path": "pull", "rows_wanted": int(want.sum()), "entries_scanned": int(entries), "bytes": int(nbytes)})
    return out


def bench_bfs(args, B, torch, dev, flush, peak):
    """DB-BFS GTEPS on the symmetrised R-MAT graph, 16 seeded sources (configs[3]); every timed
    source is compared with the oracle; per-level time, direction and algorithmic bytes for the
    first source."""
    g = wl.rmat(args.bfs_scale, 16, seed=3, values=False, symmetrise=True)
    up = lambda arr: torch.from_numpy(np.ascontiguousarray(arr)).to(dev)
    h = B.dbspmspv_create_csr(g.m, g.n, g.nnz, up(g.row_ptr), up(g.col_idx), None, B.PATTERN)
    st0 = B.dbspmspv_get_stats(h)
    srcs = wl.bfs_sources(g, 16)
    deg = np.diff(g.row_ptr)
    levels = torch.empty(g.n, dtype=torch.int32, device=dev)
    import oracle
    A = oracle.RefMatrix(g.m, g.n, g.row_ptr, g.col_idx)
    A.csc()
    times, warm_times, teps, nlev, matches, cpu_s, cpu_edges = [], [], [], [], [], 0.0, 0.0
    level_rec = None
    for s in srcs:
        ts = timed_calls(torch, lambda: B.db_bfs(h, int(s), levels), flush, 3)
        tw = timed_calls(torch, lambda: B.db_bfs(h, int(s), levels), flush, 3, warm=True)
        best = min(ts) * 1e-3
        lv = levels.cpu().numpy()
        edges = float(deg[lv >= 0].sum()) / 2.0
        times.append(best)
        warm_times.append(min(tw) * 1e-3)
        teps.append(edges / (best * 1e-3) / 1e9)
        stt = B.dbspmspv_get_stats(h)
        nlev.append(int(stt.bfs_levels))
        t0 = time.perf_counter()
        ref = oracle.ref_bfs(A, int(s))               # every timed source is compared with the oracle
        cpu_s += time.perf_counter() - t0
        cpu_edges += float(deg[ref >= 0].sum()) / 2.0
        matches.append(bool(np.array_equal(ref, lv)))
        if level_rec is None:
            nl = int(stt.bfs_levels)
            paths = [int(p) for p in stt.bfs_level_path[:nl]]
            lb = bfs_level_bytes(g, lv, paths)
            for L, rec in enumerate(lb):
                us = float(stt.bfs_level_us[L])
                rec["us"] = round(us, 1)
                rec.update(fractions(rec["bytes"], us, peak))
            total_b = float(sum(r["bytes"] for r in lb)) + 4.0 * g.n + 16.0 * ((g.n + 31) // 32)   # + initialisation of levels and masks
            level_rec = {"source": int(s), "setup_us": round(float(stt.bfs_setup_us), 1), "levels": lb, "bytes": int(total_b),
                         "call_us_l2_warm": round(min(tw), 1), "whole_call": fractions(total_b, min(tw), peak),
                         "note": "level times are device time stamps of the last (L2-warm) run of this source"}
    B.dbspmspv_destroy(h)
    hm = len(teps) / sum(1.0 / t for t in teps)
    return {"workload": f"rmat{args.bfs_scale}_sym_ef16_pattern_16sources", "gteps_harmonic_mean": round(hm, 3),
            "gteps_min": round(min(teps), 3), "gteps_max": round(max(teps), 3),
            "ms_median": round(float(np.median(times)), 4), "ms_median_l2_warm": round(float(np.median(warm_times)), 4),
            "levels": nlev, "vertices": int(g.n), "nnz": int(g.nnz),
            "sources_matching_oracle": int(sum(matches)), "sources": len(matches),
            "format_bytes": int(st0.payload_bytes + st0.csr_view_bytes + st0.csc_view_bytes + st0.segment_bytes + st0.lean_index_bytes),
            "bfs_index_bytes": int(st0.bfs_index_bytes), "roofline_first_source": level_rec,
            "cpu_baseline": {"value": round(cpu_edges / cpu_s / 1e9, 4), "unit": "GTEPS",
                             "cores": 1, "kind": "oracle", "sample": "queue BFS from each of the sources"}}


if __name__ == "__main__":
    main()
