#!/usr/bin/env python
"""Benchmark of the GMS restore / digest / verify path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 8b|mixed|tiny|kv|host70b|capture|file]
    python bench.py --impl reference ...      # the CPU oracle on this host's cores

One *step* is one pass of the whole hot path over one synthetic snapshot:
    gms_digest  (digest the preserved allocations in place)   -> gms_verify
    gms_restore (scatter the device-staged image, fused digest) -> gms_verify
(`kv`: one gms_kv_restore; `host70b`: one host-sourced gms_restore + gms_verify; `capture`: gms_capture +
gms_verify; `file`: gms_restore_fd from a file through pinned buffers).
The default workload is the Llama-3-8B-shaped weight manifest (291 tensors, 16.06 GB of random
bf16 bit patterns); image and destinations are resident in HBM when the timed region starts and are
~250x larger than L2, so no L2 flush is needed between iterations.

`value` is algorithmic HBM traffic per second over the whole step (bytes the method must read and
write: payload once for the digest pass, twice for the restore pass, plus 8 B per 4 KiB of digests
and the verify pass's 16 B per block), summed over all GPUs, timed on the device with CUDA events,
max over ranks.  `e2e` is the same metric with the snapshot image in pinned host memory:
gms_restore_staged moves it across the host link inside the timed region (copy engine -> device
ring -> restore kernel) and the verdict (mismatch count, tensor digests) is read back to the host
every step.  With N > 1 every rank restores its own
replica (the path has no exchange step): weak scaling, no data-path collective.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "restore+digest GB/s"
UNIT = "GB/s"
FALLBACK_HBM_GBS = 6650.0
DATASHEET_HBM_GBS = 8000.0
# dram__bytes_read.sum + dram__bytes_write.sum per payload byte, from the ncu captures summarised under
# profiles/: restore, digest and kv_restore measured at full size (single-pass capture of the 8B manifest and
# the 60 GB pool); capture from the small mixed-manifest case, where traffic is proportional to the payload.
NCU_DRAM_BYTES_PER_PAYLOAD_BYTE = {"restore": 2.000, "digest": 1.004, "kv_restore": 1.993, "capture": 1.983}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30, help="timed steps (a recovery restores once; long loops run power-capped)")
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["gms", "reference"], default="gms")
    ap.add_argument("--workload", choices=["8b", "mixed", "tiny", "kv", "host70b", "capture", "file"], default="8b")
    ap.add_argument("--stage-buffers", type=int, default=3, help="host70b: device ring of the copy-engine-fed variant")
    ap.add_argument("--stage-mib", type=int, default=64)
    ap.add_argument("--vmm", action="store_true", help="8b/mixed/tiny/capture/file: destinations from gms_service VMM slabs")
    ap.add_argument("--graph", action="store_true",
                    help="8b/mixed/tiny: capture the step into a CUDA graph once and time its replays (whole step only)")
    ap.add_argument("--no-l2-flush", action="store_true", help="mixed/tiny: leave L2 as the previous step left it")
    ap.add_argument("--file-dir", default="/dev/shm", help="file: where the snapshot file is written")
    ap.add_argument("--pipe-buffers", type=int, default=4)
    ap.add_argument("--pipe-mib", type=int, default=256)
    ap.add_argument("--pipe-readers", type=int, default=16)
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=12.0, help="target CPU time of the oracle sample")
    ap.add_argument("--host-gib", type=float, default=32.0, help="host70b: size of the pinned host image")
    ap.add_argument("--kv-gb", type=float, default=60.0, help="kv: size of the paged pool (a small pool is used for ncu captures)")
    return ap.parse_args()


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    """Polls SM clock and throttle reasons through NVML (read-only) while the benchmark runs."""

    def __init__(self, index: int):
        self.samples = []  # (t, sm_mhz, reasons_bitmask)
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml

            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                mhz = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                try:
                    reasons = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    reasons = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                try:
                    mem = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_MEM)
                    watts = nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0
                except Exception:
                    mem, watts = None, None
                self.samples.append((time.perf_counter(), mhz, reasons, mem, watts))
            except Exception:
                pass
            time.sleep(0.004)

    def start(self):
        if self.nv:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread:
            self._thread.join()

    def summary(self, t0: float, t1: float):
        if not self.nv:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvml_unavailable"]}
        window = "timed"
        inside = [s for s in self.samples if t0 <= s[0] <= t1]
        if len(inside) < 3:
            inside, window = self.samples, "warmup+timed"
        names = {
            0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
            0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
            0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting",
        }
        seen = 0
        for s in inside:
            seen |= s[2]
        reasons = [n for bit, n in names.items() if seen & bit and n != "gpu_idle"]
        return {
            "sm_mhz": statistics.median(s[1] for s in inside) if inside else None,
            "sm_max_mhz": self.max_mhz, "reasons": reasons, "samples": len(inside), "window": window,
            "mem_mhz": statistics.median(s[3] for s in inside) if inside and inside[0][3] is not None else None,
            "power_w": statistics.median(s[4] for s in inside) if inside and inside[0][4] is not None else None,
        }


# --------------------------------------------------------------------------- rank plumbing
def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def reduce_over_ranks(local_ms: float, local_units: float, dist=None, device=None):
    """(max over ranks of the time, sum over ranks of the units).  `dist` is torch.distributed when
    a process group is up, else None (single process)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return local_ms, local_units
    import torch

    t = torch.tensor([local_ms], dtype=torch.float64, device=device)
    u = torch.tensor([local_units], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


# --------------------------------------------------------------------------- workloads on the device
class ManifestBench:
    """digest + verify + restore + verify over a manifest workload (8b / mixed / tiny)."""

    def __init__(self, name, torch, gms, W, dev):
        self.torch, self.gms, self.W, self.dev, self.name = torch, gms, W, dev, name
        self.w = {"8b": W.llama3_8b_manifest, "mixed": W.mixed_manifest, "tiny": W.tiny_manifest}[name]()
        w = self.w
        self.image = torch.empty(w.image_bytes, dtype=torch.uint8, device=dev)
        W.fill_random_device(self.image, W.SEED_BASE + 0x100)
        self.vmm = bool(os.environ.get("GMS_BENCH_VMM"))  # set by --vmm: destinations carved from gms_service slabs
        if self.vmm:
            import numpy as np

            self.svc = gms.gms_service_create(0)  # 2 GiB slabs, dedicated slabs above that
            gms.gms_service_acquire_rw(self.svc)
            ptrs = [gms.gms_service_alloc(self.svc, max(1, int(n))) for n in w.rows["nbytes"]]
            self.slab = None
            self.entries = self._entries(0)
            self.entries["dst"] = np.array(ptrs, dtype=np.uint64)
        else:
            self.slab = torch.zeros(w.slab_bytes, dtype=torch.uint8, device=dev)
            self.entries = self._entries(self.slab.data_ptr())
        self.m = gms.gms_manifest_build(self.entries, w.image_bytes)
        self.bd = torch.zeros(max(self.m.n_blocks, 1), dtype=torch.int64, device=dev)
        self.td = torch.zeros(max(self.m.n_tensors, 1), dtype=torch.int64, device=dev)
        self.cap = 64
        self.mm = torch.zeros(2 * self.cap, dtype=torch.int64, device=dev)
        self.cnt = torch.zeros(1, dtype=torch.int64, device=dev)
        # "commit": populate the destinations once and record their digests
        gms.gms_restore(self.m, self.image, gms.SRC_DEVICE, self.bd, self.td)
        gms.gms_manifest_set_expected(self.m, self.bd)
        torch.cuda.synchronize()
        self.payload = w.payload_bytes
        self.n_chunks = gms.gms_manifest_chunk_count(self.m)
        nb = self.m.n_blocks
        self.bytes_digest = self.payload + 8 * nb + 32 * self.n_chunks
        self.bytes_restore = 2 * self.payload + 8 * nb + 32 * self.n_chunks
        self.bytes_verify = 16 * nb
        self.traffic = self.bytes_digest + self.bytes_restore + 2 * self.bytes_verify
        self.phase_names = ["digest", "verify", "restore", "verify2"]
        self.dominant = "restore"
        self.dominant_bytes = self.bytes_restore
        self.launches_per_step = None
        self.graph = None
        # a working set that L2 (126 MB) could hold between steps is flushed out before every step
        self.l2_flush = torch.zeros(256 << 20, dtype=torch.uint8, device=dev) if self.payload < (512 << 20) else None

    def use_graph(self):
        """Captures one step into a CUDA graph; later steps replay it (no per-phase times then)."""
        torch = self.torch
        n0 = self.gms.gms_kernel_launches()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            self.step()
        self.launches_per_step = self.gms.gms_kernel_launches() - n0
        self.graph = graph

    def _entries(self, base):
        import numpy as np

        w = self.w
        e = np.zeros(len(w.rows), dtype=self.gms.ENTRY_DTYPE)
        e["tensor_id"], e["src_offset"], e["nbytes"] = w.rows["tensor_id"], w.rows["src_offset"], w.rows["nbytes"]
        e["dst"] = w.rows["dst_offset"] + np.uint64(base)
        return e

    def step(self, marks=None, image=None, kind=None):
        g, m = self.gms, self.m
        if self.graph is not None and image is None:
            if marks: marks[0].record()
            self.graph.replay()
            if marks:
                for e in marks[1:]: e.record()
            return
        if marks: marks[0].record()
        g.gms_digest(m, self.bd, self.td)
        if marks: marks[1].record()
        g.gms_verify(m, self.bd, self.mm, self.cap, self.cnt)
        if marks: marks[2].record()
        g.gms_restore(m, self.image if image is None else image, g.SRC_DEVICE if kind is None else kind, self.bd, self.td)
        if marks: marks[3].record()
        g.gms_verify(m, self.bd, self.mm, self.cap, self.cnt)
        if marks: marks[4].record()

    def check(self):
        self.torch.cuda.synchronize()
        assert int(self.cnt.item()) == 0, "verify reported mismatches on an intact restore"
        assert self.gms.gms_last_device_status(self.m) == 0

    def config(self):
        return {"workload": f"{self.w.name}: {len(self.w.rows)} tensors, {self.payload} B payload, "
                            f"{self.m.n_blocks} digest blocks, {self.n_chunks} chunks",
                "step": "gms_digest + gms_verify + gms_restore(device image) + gms_verify",
                "destinations": "gms_service VMM slabs (2 GiB, first fit)" if self.vmm else "carved from one cudaMalloc slab",
                "l2": "inputs larger than L2 (no flush)" if self.payload >= (512 << 20) else
                      ("L2 flushed before every step (256 MiB read+write, outside the phase events); ms_per_step = sum of phases"
                       if self.l2_flush is not None else "working set near L2 size; not flushed"),
                "payload_bytes": self.payload}


class CaptureBench(ManifestBench):
    """gms_capture of the 8B manifest (allocations -> packed device image, fused digest) + gms_verify."""

    def __init__(self, torch, gms, W, dev):
        super().__init__("8b", torch, gms, W, dev)
        self.phase_names = ["capture", "verify"]
        self.dominant, self.dominant_bytes = "capture", self.bytes_restore
        self.traffic = self.bytes_restore + self.bytes_verify

    def step(self, marks=None, image=None, kind=None):
        g, m = self.gms, self.m
        if marks: marks[0].record()
        g.gms_capture(m, self.image, g.SRC_DEVICE, self.bd, self.td)
        if marks: marks[1].record()
        g.gms_verify(m, self.bd, self.mm, self.cap, self.cnt)
        if marks: marks[2].record()

    def config(self):
        c = super().config()
        c["step"] = "gms_capture(device image) + gms_verify"
        return c


class KvBench:
    """gms_kv_restore of a seeded 10% of a paged KV pool."""

    def __init__(self, torch, gms, W, dev, pool_bytes=60e9):
        self.torch, self.gms = torch, gms
        k = self.k = W.kv_pool_workload(pool_bytes=pool_bytes)
        self.pool = torch.empty(k.pool_bytes, dtype=torch.uint8, device=dev)
        W.fill_random_device(self.pool, W.SEED_BASE + 0x200)
        self.image = torch.empty(k.image_bytes, dtype=torch.uint8, device=dev)
        W.fill_random_device(self.image, W.SEED_BASE + 0x201)
        self.ids = torch.from_numpy(k.ids).to(dev)
        kk = k.block_bytes // 4096
        self.bd = torch.zeros(len(k.ids) * k.n_planes * kk, dtype=torch.int64, device=dev)
        self.kd = torch.zeros(len(k.ids), dtype=torch.int64, device=dev)
        self.st = torch.zeros(4, dtype=torch.int64, device=dev)
        self.desc = gms.KvPool(base=self.pool.data_ptr(), plane_stride=k.plane_stride, block_stride=k.block_stride,
                               n_planes=k.n_planes, n_blocks=k.n_blocks, block_bytes=k.block_bytes)
        self.payload = k.payload_bytes
        self.bytes_restore = 2 * self.payload + 8 * self.bd.numel()
        self.bytes_digest = self.payload + 8 * self.bd.numel()
        self.bytes_verify = 16 * self.bd.numel()
        self.traffic = self.bytes_restore + self.bytes_digest + self.bytes_verify
        self.phase_names = ["kv_restore", "kv_digest", "kv_verify"]
        self.dominant, self.dominant_bytes = "kv_restore", self.bytes_restore
        # digests of the restore, against which the in-place digests are verified (allocation-free flat verify)
        self.bd_restore = torch.zeros_like(self.bd)
        self.mm = torch.zeros(2 * 64, dtype=torch.int64, device=dev)
        self.cnt = torch.zeros(1, dtype=torch.int64, device=dev)
        self.flat_verify = self.bd.numel() <= 4194304  # the entry point's fixed scratch

    def step(self, marks=None, image=None, kind=None):
        g, k = self.gms, self.k
        if marks: marks[0].record()
        g.gms_kv_restore(self.desc, self.image, k.img_plane_stride, k.img_slot_stride, g.SRC_DEVICE, self.ids, len(k.ids),
                         self.bd_restore, self.kd, self.st)
        if marks: marks[1].record()
        g.gms_kv_digest(self.desc, self.ids, len(k.ids), self.bd, self.kd, self.st)
        if marks: marks[2].record()
        if self.flat_verify:
            g.gms_verify_flat_noalloc(self.bd, self.bd_restore, self.bd.numel(), 0, self.mm, 64, self.cnt)
        if marks: marks[3].record()

    def check(self):
        self.torch.cuda.synchronize()
        assert self.st[:2].tolist() == [0, 0]
        assert int(self.cnt.item()) == 0, "in-place KV digests differ from the ones the restore reported"

    def config(self):
        k = self.k
        return {"workload": f"{k.name}: pool {k.pool_bytes} B, {len(k.ids)} of {k.n_blocks} blocks selected, {self.payload} B moved",
                "step": "gms_kv_restore(device image) + gms_kv_digest(the same blocks in place) + gms_verify_flat_noalloc", "l2": "inputs larger than L2 (no flush)", "payload_bytes": self.payload}


def event_list(torch, n):
    return [torch.cuda.Event(enable_timing=True) for _ in range(n)]


PHASE_STATS = {}  # per-phase median and best of the last timed_steps() call (ms)


def timed_steps(torch, bench, steps, dist=None, **step_kw):
    """Times `steps` steps with CUDA events on the current stream; returns (total ms, per-phase mean ms).

    If the bench object carries an `l2_flush` tensor (working sets that would otherwise sit in L2), it is
    rewritten before every step, outside every phase's event pair, and the total is the sum of the phases."""
    flush = getattr(bench, "l2_flush", None)
    n_marks = len(bench.phase_names) + 1
    marks = [event_list(torch, n_marks) for _ in range(steps)]
    e0, e1 = event_list(torch, 2)
    torch.cuda.synchronize()
    if dist is not None and dist.is_initialized():
        dist.barrier()
        torch.cuda.synchronize()
    t0 = time.perf_counter()
    e0.record()
    for i in range(steps):
        if flush is not None:
            flush.add_(1)  # read + write of a buffer twice the size of L2
        bench.step(marks[i], **step_kw)
    e1.record()
    torch.cuda.synchronize()
    t1 = time.perf_counter()
    if dist is not None and dist.is_initialized():
        dist.barrier()
        torch.cuda.synchronize()
    total = e0.elapsed_time(e1)
    phases = {}
    PHASE_STATS.clear()
    for p, name in enumerate(bench.phase_names):
        ts = [marks[i][p].elapsed_time(marks[i][p + 1]) for i in range(steps)]
        phases[name] = statistics.fmean(ts)
        PHASE_STATS[name] = {"median": statistics.median(ts), "best": min(ts)}
    if flush is not None:
        total = sum(phases.values()) * steps
    return total, phases, (t0, t1)


# --------------------------------------------------------------------------- CPU oracle legs
def oracle_sample_rows(w, max_bytes):
    """Prefix of the workload's tensors (record order) totalling at most max_bytes (at least one tensor)."""
    rows, used = [], 0
    for r in w.rows:
        nb = int(r["nbytes"])
        if rows and used + nb > max_bytes:
            break
        rows.append(r)
        used += nb
        if used >= max_bytes:
            break
    return rows, used


def oracle_step(oracle, rec, image, slab, expected):
    """The step, on the CPU: digest + verify + restore + verify.  Returns mismatch count (0)."""
    _, bd, _ = oracle.digest(rec, slab)
    c1, _ = oracle.verify(rec, bd, expected, 64)
    _, bd, _ = oracle.restore(rec, image, slab)
    c2, _ = oracle.verify(rec, bd, expected, 64)
    return c1 + c2


def make_oracle_sample(oracle, W, w, sample_bytes, image_fetch):
    """Builds host copies for a prefix sample.  image_fetch(lo, hi) returns image bytes [lo, hi) as numpy."""
    import numpy as np

    rows, used = oracle_sample_rows(w, sample_bytes)
    # re-pack the sample densely: sources keep their bytes, destinations are packed on the host
    rec_rows, src_parts, off = [], [], 0
    for r in rows:
        nb = int(r["nbytes"])
        rec_rows.append((int(r["tensor_id"]), off, off, nb))
        src_parts.append(image_fetch(int(r["src_offset"]), int(r["src_offset"]) + nb))
        off += (nb + 15) // 16 * 16
        pad = off - (rec_rows[-1][1] + nb)
        if pad:
            src_parts.append(np.zeros(pad, np.uint8))
    image = np.concatenate(src_parts) if src_parts else np.zeros(16, np.uint8)
    slab = np.zeros(max(off, 16), np.uint8)
    rec = oracle.make_record(rec_rows)
    _, expected, _ = oracle.restore(rec, image, slab)  # "commit" on the host (untimed)
    return rec, image, slab, expected, used, len(rows)


def cpu_baseline(args, bench, W, torch):
    """Times the oracle, as it stands, on a bounded prefix sample of the same workload (1 thread)."""
    from oracle import gms_oracle as oracle

    w = bench.w
    fetch = lambda lo, hi: bench.image[lo:hi].cpu().numpy()
    # calibrate on ~32 MB, then size the sample for about args.cpu_seconds
    rec, image, slab, expected, used, _ = make_oracle_sample(oracle, W, w, 32 << 20, fetch)
    t = time.perf_counter()
    oracle_step(oracle, rec, image, slab, expected)
    per_byte = (time.perf_counter() - t) / max(used, 1)
    target = int(min(max(args.cpu_seconds / per_byte, 32 << 20), 8 << 30))
    rec, image, slab, expected, used, n = make_oracle_sample(oracle, W, w, target, fetch)
    t = time.perf_counter()
    bad = oracle_step(oracle, rec, image, slab, expected)
    dt = time.perf_counter() - t
    assert bad == 0
    nb = int(sum((int(r[3]) + 4095) // 4096 for r in rec))
    traffic = 3 * used + 16 * nb + 2 * 16 * nb
    out = {"value": traffic / dt / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
           "sample": f"first {n} tensors of the manifest ({used} B payload), one step = digest+verify+restore+verify, "
                     f"{dt:.2f} s on 1 of {os.cpu_count()} host cores"}
    # the same oracle functions on all host cores: the sample's tensors are dealt out to threads (the oracle itself
    # is single-threaded and untouched; ctypes releases the GIL), each thread works on its own sub-record
    import concurrent.futures as cf

    cores = os.cpu_count() or 1
    order = sorted(range(len(rec)), key=lambda i: -int(rec[i]["nbytes"]))
    loads, groups = [0] * cores, [[] for _ in range(cores)]
    for i in order:  # largest first onto the least loaded thread
        k = loads.index(min(loads))
        groups[k].append(i)
        loads[k] += int(rec[i]["nbytes"])
    shards = []
    for g in groups:
        if g:
            sub = rec[sorted(g)]
            _, exp_sub, _ = oracle.digest(sub, slab)  # slab holds the restored bytes: these are the recorded digests
            shards.append((sub, exp_sub))
    with cf.ThreadPoolExecutor(len(shards)) as ex:
        t = time.perf_counter()
        bad = sum(ex.map(lambda s: oracle_step(oracle, s[0], image, slab, s[1]), shards))
        dt_all = time.perf_counter() - t
    assert bad == 0
    out["all_cores"] = {"value": traffic / dt_all / 1e9, "unit": UNIT, "cores": len(shards), "seconds": dt_all}
    return out


def cpu_baseline_kv(bench, planes=16):
    """The oracle's kv_restore (1 thread) on the first `planes` planes of the same pool shape, image and id list."""
    import numpy as np

    from oracle import gms_oracle as oracle

    k = bench.k
    planes = min(planes, k.n_planes)
    image = bench.image[: planes * k.img_plane_stride].cpu().numpy()
    pool = np.empty(planes * k.plane_stride, dtype=np.uint8)  # only the selected blocks are ever touched
    t = time.perf_counter()
    rc, bd, kd, skipped = oracle.kv_restore(pool, k.plane_stride, k.block_stride, planes, k.n_blocks, k.block_bytes, image,
                                            k.img_plane_stride, k.img_slot_stride, k.ids)
    rc2, bd2, kd2, _ = oracle.kv_digest(pool, k.plane_stride, k.block_stride, planes, k.n_blocks, k.block_bytes, k.ids)
    dt = time.perf_counter() - t
    assert rc == 0 and rc2 == 0 and skipped == 0 and (bd2 == bd).all() and (kd2 == kd).all()
    moved = planes * len(k.ids) * k.block_bytes
    return {"value": (3 * moved + 16 * bd.size) / dt / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"kv_restore + kv_digest on the first {planes} of {k.n_planes} planes of the same pool, image and id list ({moved} B moved), "
                      f"{dt:.2f} s on 1 of {os.cpu_count()} host cores"}


def reference_arm(args):
    """`--impl reference`: the oracle on this host's cores, same metric, bounded sample per step."""
    rank, _, world = dist_env()
    if rank != 0:
        return
    import numpy as np

    from oracle import gms_oracle as oracle
    from paper_2609_25451_b200 import workloads as W

    w = {"8b": W.llama3_8b_manifest, "mixed": W.mixed_manifest, "tiny": W.tiny_manifest}.get(args.workload, W.llama3_8b_manifest)()
    rng_image = {}

    def fetch(lo, hi):  # synthetic bytes generated on the host for the sampled range only
        key = (lo, hi)
        if key not in rng_image:
            rng_image[key] = W.random_bytes_host(hi - lo, seed=(W.SEED_BASE + lo) & 0x7FFFFFFF)
        return rng_image[key]

    per_step_s = min(3.0, 150.0 / max(args.steps + args.warmup, 1))
    rec, image, slab, expected, used, _ = make_oracle_sample(oracle, W, w, 16 << 20, fetch)
    t = time.perf_counter()
    oracle_step(oracle, rec, image, slab, expected)
    per_byte = (time.perf_counter() - t) / max(used, 1)
    target = int(min(max(per_step_s / per_byte, 4 << 20), 4 << 30))
    rec, image, slab, expected, used, n = make_oracle_sample(oracle, W, w, target, fetch)
    for _ in range(args.warmup):
        oracle_step(oracle, rec, image, slab, expected)
    t = time.perf_counter()
    for _ in range(args.steps):
        assert oracle_step(oracle, rec, image, slab, expected) == 0
    dt = time.perf_counter() - t
    nb = int(sum((int(r[3]) + 4095) // 4096 for r in rec))
    traffic = (3 * used + 48 * nb) * args.steps
    value = traffic / dt / 1e9
    sample = f"each step: first {n} tensors of {w.name} ({used} B payload), digest+verify+restore+verify, 1 thread"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / max(args.steps, 1) * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u64", "data": "synthetic",
        "config": {"workload": f"{w.name} (bounded sample per step)", "payload_bytes": used},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------- host-sourced legs
def host_image_of(torch, gms, dev_image):
    """Pinned, device-mapped host copy of a device image.  Returns (host_ptr, device_view, cpu tensor)."""
    import numpy as np  # noqa: F401

    n = dev_image.numel()
    hptr, dview, arr = gms.gms_host_image_alloc(n)
    cpu = torch.from_numpy(arr)
    step = 1 << 30
    for a in range(0, n, step):
        cpu[a:a + step].copy_(dev_image[a:a + step])
    torch.cuda.synchronize()
    return hptr, dview, cpu


def per_tensor_memcpy_yardstick(torch, bench, reps=3):
    """The launch-per-tensor way of moving the same payload (no digest): one device-to-device cudaMemcpyAsync per
    manifest entry on one stream, issued through ctypes.  Returns (best device-timed ms, best host-issue ms, calls)."""
    import ctypes

    try:
        rt = ctypes.CDLL("libcudart.so.12")  # the runtime torch has already loaded
    except OSError:
        return None
    f = rt.cudaMemcpyAsync
    f.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int, ctypes.c_void_p]
    f.restype = ctypes.c_int
    base = bench.image.data_ptr()
    e = bench.entries
    calls = [(int(d), base + int(s), int(n)) for d, s, n in zip(e["dst"], e["src_offset"], e["nbytes"]) if n]
    stream = torch.cuda.current_stream().cuda_stream
    best_dev, best_host = float("inf"), float("inf")
    for _ in range(reps):
        a, b = event_list(torch, 2)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        a.record()
        for d, s, n in calls:
            if f(d, s, n, 3, stream):  # 3 = cudaMemcpyDeviceToDevice
                return None
        b.record()
        t1 = time.perf_counter()
        torch.cuda.synchronize()
        best_dev, best_host = min(best_dev, a.elapsed_time(b)), min(best_host, (t1 - t0) * 1e3)
    return best_dev, best_host, len(calls)


def h2d_yardstick(torch, cpu_tensor, dev_tensor, reps=3):
    """Plain cudaMemcpyAsync host->device of the whole pinned image (torch copy_), best of reps, GB/s."""
    best = None
    for _ in range(reps + 1):
        a, b = event_list(torch, 2)
        a.record()
        dev_tensor.copy_(cpu_tensor, non_blocking=True)
        b.record()
        torch.cuda.synchronize()
        ms = a.elapsed_time(b)
        best = ms if best is None else min(best, ms)
    return cpu_tensor.numel() / best / 1e6


def main():
    args = parse_args()
    if args.impl == "reference":
        reference_arm(args)
        return
    if args.vmm:
        os.environ["GMS_BENCH_VMM"] = "1"
    rank, local_rank, world = dist_env()
    import torch
    import torch.distributed as dist

    from paper_2609_25451_b200 import gms
    from paper_2609_25451_b200 import workloads as W

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the data path has no CPU implementation")
    gms.lib()  # fail loudly if libgms.so is missing
    torch.cuda.set_device(local_rank)
    gms.gms_set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    use_dist = world > 1
    if use_dist:
        dist.init_process_group("nccl", device_id=dev)
    d = dist if use_dist else None

    sampler = ClockSampler(local_rank)
    if args.workload == "kv":
        bench = KvBench(torch, gms, W, dev, pool_bytes=args.kv_gb * 1e9)
    elif args.workload in ("host70b", "file"):
        bench = None
    elif args.workload == "capture":
        bench = CaptureBench(torch, gms, W, dev)
    else:
        bench = ManifestBench(args.workload, torch, gms, W, dev)

    if args.workload == "host70b":
        run_host70b(args, torch, gms, W, dev, sampler, rank)
        return
    if args.workload == "file":
        run_file(args, torch, gms, W, dev, sampler, rank)
        return

    if args.no_l2_flush and getattr(bench, "l2_flush", None) is not None:
        bench.l2_flush = None
    for _ in range(max(args.warmup, 3)):
        bench.step()
    bench.check()
    graphed = args.graph and type(bench) is ManifestBench
    if graphed:
        bench.use_graph()
        for _ in range(3):
            bench.step()
        bench.check()
    launches0 = gms.gms_kernel_launches()
    sampler.start()
    total_ms, phases, (t0, t1) = timed_steps(torch, bench, args.steps, d)
    sampler.stop()
    launches = gms.gms_kernel_launches() - launches0
    if graphed:  # replays do not pass through the library's launch counter
        launches = bench.launches_per_step * args.steps
        phases = {"step": total_ms / args.steps}
    bench.check()
    clocks = sampler.summary(t0, t1)

    max_ms, sum_traffic = reduce_over_ranks(total_ms, float(bench.traffic) * args.steps, d, dev)
    value = sum_traffic / max_ms / 1e6
    peak, peak_kind = measured_peak()
    if graphed:  # one event pair around each replay: the whole step's bytes over the whole step's time
        achieved = bench.traffic / phases["step"] / 1e6
        roofline = {
            "kernel": "whole step replayed from a CUDA graph (digest + verify + restore + verify)",
            "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
            "peak_kind": f"of {peak_kind}", "frac_of_datasheet_8TBps": achieved / DATASHEET_HBM_GBS,
            "algorithmic_bytes_per_launch": bench.traffic, "traffic": None,
        }
    else:
        dom_ms = phases[bench.dominant]
        achieved = bench.dominant_bytes / dom_ms / 1e6
        ratio = NCU_DRAM_BYTES_PER_PAYLOAD_BYTE.get(bench.dominant)
        roofline = {
            "kernel": f"gms_{'kv_' if bench.dominant == 'kv_restore' else ''}stream_kernel ({bench.dominant}; duration = the "
                      "call's events, incl. its one-block prologue)",
            "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
            "peak_kind": f"of {peak_kind}", "frac_of_datasheet_8TBps": achieved / DATASHEET_HBM_GBS,
            "algorithmic_bytes_per_launch": bench.dominant_bytes,
            "traffic": (ratio * bench.payload) if ratio else None,
        }

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": max_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "u64", "data": "synthetic", "config": bench.config(), "roofline": roofline, "clocks": clocks,
        "gpu_launches": int(launches),
        "phases_ms": phases, "phases_ms_median_best": {} if graphed else dict(PHASE_STATS),
        "geometry": gms.gms_launch_geometry(),
    }
    if type(bench) is ManifestBench and "restore" in phases:
        y = per_tensor_memcpy_yardstick(torch, bench)
        if y:
            line["per_tensor_memcpy"] = {
                "ms": y[0], "host_issue_ms": y[1], "calls": y[2], "payload_gbs": bench.payload / y[0] / 1e6,
                "restore_speedup": y[0] / phases["restore"],
                "note": "one cudaMemcpyAsync D2D per tensor on one stream, no digest (the launch-per-tensor yardstick)"}
    if graphed:
        line["config"]["launch"] = f"CUDA graph replay ({bench.launches_per_step} kernel nodes per step)"
    if "restore" in phases:
        line["restore_s"] = phases["restore"] / 1e3
        line["restore_payload_gbs"] = bench.payload / phases["restore"] / 1e6
        line["digest_read_gbs"] = bench.bytes_digest / phases["digest"] / 1e6
        line["digest_frac_of_peak"] = line["digest_read_gbs"] / peak

    # ---- end to end: snapshot image in pinned host memory, verdict read back every step
    if not args.no_e2e and type(bench) is ManifestBench:
        hptr, dview, cpu = host_image_of(torch, gms, bench.image)
        h2d_gbs = h2d_yardstick(torch, cpu, bench.image)
        pin_cnt = torch.zeros(1, dtype=torch.int64).pin_memory()
        pin_td = torch.zeros(bench.td.numel(), dtype=torch.int64).pin_memory()

        class E2E:
            phase_names = bench.phase_names + ["readback"]

            @staticmethod
            def step(marks=None):
                # the step with a HOST image: the pinned image crosses the link inside gms_restore_staged
                # (copy engine -> device ring -> restore kernel); results come back to pinned host memory
                g, m = gms, bench.m
                if marks: marks[0].record()
                g.gms_digest(m, bench.bd, bench.td)
                if marks: marks[1].record()
                g.gms_verify(m, bench.bd, bench.mm, bench.cap, bench.cnt)
                if marks: marks[2].record()
                g.gms_restore_staged(m, stage, hptr, bench.bd, bench.td)
                if marks: marks[3].record()
                g.gms_verify(m, bench.bd, bench.mm, bench.cap, bench.cnt)
                if marks: marks[4].record()
                pin_cnt.copy_(bench.cnt, non_blocking=True)
                pin_td.copy_(bench.td, non_blocking=True)
                if marks: marks[5].record()

        stage = gms.gms_stage_create(args.stage_buffers, args.stage_mib << 20)
        E2E.step()
        torch.cuda.synchronize()
        e_ms, e_ph, _ = timed_steps(torch, E2E, max(args.e2e_steps, 1), d)
        assert int(pin_cnt.item()) == 0
        e_max, e_traffic = reduce_over_ranks(e_ms, float(bench.traffic) * max(args.e2e_steps, 1), d, dev)
        # for comparison: the same restore with kernel-issued reads of the mapped image (no copy engine)
        ma, mb = event_list(torch, 2)
        ma.record()
        gms.gms_restore(bench.m, dview, gms.SRC_HOST_MAPPED, bench.bd, bench.td)
        mb.record()
        torch.cuda.synchronize()
        mapped_gbs = bench.payload / ma.elapsed_time(mb) / 1e6
        line["e2e"] = {
            "value": e_traffic / e_max / 1e6, "unit": UNIT, "h2d_bytes_per_step": bench.payload,
            "d2h_bytes_per_step": 8 + 8 * bench.td.numel(), "steps": max(args.e2e_steps, 1),
            "ms_per_step": e_max / max(args.e2e_steps, 1),
            "call": f"gms_restore_staged ({args.stage_buffers} x {args.stage_mib} MiB device ring)",
            "host_restore_gbs": bench.payload / e_ph["restore"] / 1e6, "h2d_memcpy_gbs": h2d_gbs,
            "host_restore_frac_of_memcpy": bench.payload / e_ph["restore"] / 1e6 / h2d_gbs,
            "host_mapped_restore_gbs": mapped_gbs, "host_mapped_frac_of_memcpy": mapped_gbs / h2d_gbs,
        }
        torch.cuda.synchronize()
        stage.close()
        gms.gms_host_image_free(hptr)
    elif not args.no_e2e:
        line["e2e"] = None

    if rank == 0 and world == 1 and not args.no_cpu_baseline and type(bench) is ManifestBench:
        line["cpu_baseline"] = cpu_baseline(args, bench, W, torch)
    elif rank == 0 and world == 1 and not args.no_cpu_baseline and type(bench) is KvBench:
        line["cpu_baseline"] = cpu_baseline_kv(bench)

    if rank == 0:
        print(json.dumps(line), flush=True)
    if use_dist:
        dist.barrier()
        dist.destroy_process_group()


def run_file(args, torch, gms, W, dev, sampler, rank):
    """Storage-fed restore of the 8B manifest: file -> ring of pinned buffers -> device (gms_restore_fd),
    against (a) the same reader pool filling one pinned buffer with nothing consuming it and (b) the
    host-mapped restore of a fully resident pinned image."""
    import concurrent.futures as cf

    bench = ManifestBench("8b", torch, gms, W, dev)
    w = bench.w
    path = os.path.join(args.file_dir, f"gms_bench_image_{os.getpid()}.bin")
    n_buf, buf_bytes, n_readers = args.pipe_buffers, args.pipe_mib << 20, args.pipe_readers
    try:
        with open(path, "wb") as f:
            for a in range(0, w.image_bytes, 1 << 30):
                f.write(bench.image[a:a + (1 << 30)].cpu().numpy().tobytes())
        fd = os.open(path, os.O_RDONLY)
        # (a) read-only yardstick: the same slicing, one pinned buffer, no GPU work
        hptr, _, arr = gms.gms_host_image_alloc(buf_bytes)
        mv = memoryview(arr)
        slice_b = max(1 << 20, buf_bytes // n_readers)

        def read_all():
            with cf.ThreadPoolExecutor(n_readers) as ex:
                for lo in range(0, w.image_bytes, buf_bytes):
                    n = min(buf_bytes, w.image_bytes - lo)
                    futs = [ex.submit(os.preadv, fd, [mv[o:min(o + slice_b, n)]], lo + o) for o in range(0, n, slice_b)]
                    for fu in futs:
                        fu.result()

        read_all()
        t = time.perf_counter()
        read_all()
        read_gbs = w.image_bytes / (time.perf_counter() - t) / 1e9
        gms.gms_host_image_free(hptr)
        pipe = gms.gms_pipe_create(n_buf, buf_bytes, n_readers)
        gms.gms_restore_fd(bench.m, pipe, fd, 0, bench.bd, bench.td)
        steps = max(1, min(args.steps, 5))
        sampler.start()
        t0 = time.perf_counter()
        stats = [gms.gms_restore_fd(bench.m, pipe, fd, 0, bench.bd, bench.td) for _ in range(steps)]
        t1 = time.perf_counter()
        sampler.stop()
        gms.gms_verify(bench.m, bench.bd, bench.mm, bench.cap, bench.cnt)
        bench.check()
        best = min(s["total_seconds"] for s in stats)
        gbs = w.payload_bytes / best / 1e9
        line = {
            "metric": "file-sourced restore+digest GB/s", "value": gbs, "unit": UNIT, "n_gpus": 1, "steps": steps, "warmup": 1,
            "ms_per_step": best * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u64",
            "data": "synthetic",
            "config": {"workload": f"{w.name}: {w.payload_bytes} B read from {args.file_dir} through {n_buf} x {args.pipe_mib} MiB "
                                   f"pinned buffers, {n_readers} reader threads", "step": "gms_restore_fd (wall clock, synchronous call)",
                       "l2": "inputs larger than L2 (no flush)"},
            "roofline": {"bound": "storage_read", "achieved": gbs, "peak": read_gbs, "unit": "GB/s", "frac": gbs / read_gbs,
                         "peak_kind": "same file, same reader threads and slicing, into one pinned buffer with no consumer", "traffic": None},
            "pipe_stats_best": min(stats, key=lambda s: s["total_seconds"]),
            "clocks": sampler.summary(t0, t1), "gpu_launches": int(stats[0]["windows"]) * 2 * steps,
        }
        if rank == 0:
            print(json.dumps(line), flush=True)
        pipe.close()
        os.close(fd)
    finally:
        if os.path.exists(path):
            os.remove(path)


def run_host70b(args, torch, gms, W, dev, sampler, rank):
    """Host-sourced restore of a Llama-3-70B TP8 shard manifest from a pinned, mapped host image,
    against a plain cudaMemcpyAsync of the same bytes from the same allocation."""
    import numpy as np

    image_bytes = int(args.host_gib * (1 << 30)) // 16 * 16
    w = W.llama3_70b_tp8_shard_manifest(image_bytes=image_bytes)
    hptr, dview, arr = gms.gms_host_image_alloc(w.image_bytes)
    cpu = torch.from_numpy(arr)
    scratch = torch.empty(1 << 30, dtype=torch.uint8, device=dev)
    for i, a in enumerate(range(0, w.image_bytes, 1 << 30)):  # random bits made on the GPU, copied to the host image
        n = min(1 << 30, w.image_bytes - a)
        W.fill_random_device(scratch[:n], W.SEED_BASE + 0x500 + i)
        cpu[a:a + n].copy_(scratch[:n])
    slab = torch.zeros(w.slab_bytes, dtype=torch.uint8, device=dev)
    e = np.zeros(len(w.rows), dtype=gms.ENTRY_DTYPE)
    e["tensor_id"], e["src_offset"], e["nbytes"] = w.rows["tensor_id"], w.rows["src_offset"], w.rows["nbytes"]
    e["dst"] = w.rows["dst_offset"] + np.uint64(slab.data_ptr())
    m = gms.gms_manifest_build(e, w.image_bytes)
    bd = torch.zeros(m.n_blocks, dtype=torch.int64, device=dev)
    td = torch.zeros(m.n_tensors, dtype=torch.int64, device=dev)
    cnt = torch.zeros(1, dtype=torch.int64, device=dev)
    mm = torch.zeros(128, dtype=torch.int64, device=dev)
    # yardstick: one cudaMemcpyAsync of the payload-sized prefix of the same pinned allocation
    dst = slab[: min(w.payload_bytes, slab.numel())]
    h2d = h2d_yardstick(torch, cpu[: dst.numel()], dst, reps=5)
    h2d_1gib = h2d_yardstick(torch, cpu[: 1 << 30], dst[: 1 << 30], reps=5) if dst.numel() >= (1 << 30) else None
    gms.gms_restore(m, dview, gms.SRC_HOST_MAPPED, bd, td)
    gms.gms_manifest_set_expected(m, bd)
    torch.cuda.synchronize()
    steps = max(1, min(args.steps, 5))
    sampler.start()
    ev = [event_list(torch, 3) for _ in range(steps)]
    t0 = time.perf_counter()
    for i in range(steps):
        ev[i][0].record()
        gms.gms_restore(m, dview, gms.SRC_HOST_MAPPED, bd, td)
        ev[i][1].record()
        gms.gms_verify(m, bd, mm, 64, cnt)
        ev[i][2].record()
    torch.cuda.synchronize()
    t1 = time.perf_counter()
    sampler.stop()
    assert int(cnt.item()) == 0 and gms.gms_last_device_status(m) == 0
    r_ms = min(ev[i][0].elapsed_time(ev[i][1]) for i in range(steps))
    tot = statistics.fmean(ev[i][0].elapsed_time(ev[i][2]) for i in range(steps))
    gbs = w.payload_bytes / r_ms / 1e6
    line = {
        "metric": "host-sourced restore+digest GB/s", "value": w.payload_bytes / tot / 1e6, "unit": UNIT, "n_gpus": 1,
        "steps": steps, "warmup": 1, "ms_per_step": tot, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "u64", "data": "synthetic",
        "config": {"workload": f"{w.name}: {len(w.rows)} tensors, {w.payload_bytes} B payload in a {w.image_bytes} B pinned mapped host image",
                   "step": "gms_restore(host-mapped image) + gms_verify", "l2": "inputs larger than L2 (no flush)"},
        "roofline": {"bound": "host_link", "achieved": gbs, "peak": h2d, "unit": "GB/s", "frac": gbs / h2d,
                     "peak_kind": "cudaMemcpyAsync H2D of the whole payload from the same pinned allocation, same run, best of 5",
                     "h2d_memcpy_1gib_gbs": h2d_1gib, "traffic": None},
        "clocks": sampler.summary(t0, t1), "gpu_launches": steps * 5,
    }
    # the copy-engine-fed variant of the same restore (device ring, windows ordered by stream events)
    stage = gms.gms_stage_create(args.stage_buffers, args.stage_mib << 20)
    gms.gms_restore_staged(m, stage, hptr, bd, td)
    torch.cuda.synchronize()
    ev = [event_list(torch, 2) for _ in range(steps)]
    for i in range(steps):
        ev[i][0].record()
        gms.gms_restore_staged(m, stage, hptr, bd, td)
        ev[i][1].record()
    gms.gms_verify(m, bd, mm, 64, cnt)
    torch.cuda.synchronize()
    assert int(cnt.item()) == 0 and gms.gms_last_device_status(m) == 0
    s_ms = min(ev[i][0].elapsed_time(ev[i][1]) for i in range(steps))
    s_gbs = w.payload_bytes / s_ms / 1e6
    line["staged"] = {"step": f"gms_restore_staged ({args.stage_buffers} x {args.stage_mib} MiB device ring, copy engine on the link)",
                      "achieved": s_gbs, "peak": h2d, "unit": "GB/s", "frac": s_gbs / h2d, "ms": s_ms}
    shard = 17640718336  # one 70B TP8 shard; the image holds about 1.95 of them
    line["one_shard_restore_s"] = {"mapped": shard / gbs / 1e9, "staged": shard / s_gbs / 1e9, "memcpy_h2d": shard / h2d / 1e9}
    if rank == 0:
        print(json.dumps(line), flush=True)
    torch.cuda.synchronize()
    stage.close()
    m.close()
    gms.gms_host_image_free(hptr)


if __name__ == "__main__":
    main()
