#!/usr/bin/env python
"""Benchmark of the GMS restore / digest / verify path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W]          # headline (8B manifest) + all five configurations
    python bench.py --workload 8b|mixed|tiny|kv|host70b|capture|file ...   # one workload only
    python bench.py --impl reference [--workload ...]            # the CPU oracle on this host's cores

One *step* is one pass of the whole hot path over one synthetic snapshot:
    gms_digest_verify  (digest the preserved allocations in place, compare with the recorded digests)
    gms_restore_verify (scatter the device-staged image, fused digest, compare)
(`--unfused` times the same work as four calls: gms_digest, gms_verify, gms_restore, gms_verify;
`kv`: gms_kv_restore + gms_kv_digest + gms_kv_verify; `host70b`: host-sourced gms_restore + gms_verify, mapped and
copy-engine-fed; `capture`: gms_capture + gms_verify; `file`: gms_restore_fd from a file through pinned buffers).

The headline workload is the Llama-3-8B-shaped weight manifest (291 tensors, 16.06 GB of random bf16 bit
patterns); image and destinations are resident in HBM when the timed region starts and are ~250x larger than L2,
so no L2 flush is needed between iterations.  With no --workload and one GPU, the same process then measures the
other four configurations one after another (tiny, mixed, the 60 GB KV pool, the 32 GiB host image), freeing each
before the next, and reports all five under `configs`, each with its phases, roofline fraction, clocks, CPU
baseline and a parity flag.

`value` is algorithmic HBM traffic per second over the whole step (bytes the method must read and write: payload
once for the digest pass, twice for the restore pass, plus 8 B per 4 KiB of digests written and 8 B read for the
compare, and 32 B per chunk descriptor), summed over all GPUs, timed on the device with CUDA events, max over
ranks.  `e2e` is the same step with the snapshot image in pinned host memory: gms_restore_staged moves it across
the host link inside the timed region (copy engine -> device ring -> restore kernel) and the verdict (mismatch
count, tensor digests) is read back to the host every step.  With N > 1 every rank restores its own replica (the
path has no exchange step): weak scaling, no data-path collective; only the headline workload runs then.
"""
from __future__ import annotations

import argparse
import gc
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
# dram__bytes_read.sum + dram__bytes_write.sum per payload byte, from the ncu captures summarised under profiles/
# (small cases of the same kernels: a 1 GB manifest of the 8B structure, a 6 GB KV pool).  Traffic grows in
# proportion to the payload, except that the write side of a small case is short by what L2 still holds when the
# kernel ends (about 50 MB); the figures are used as they were measured.  Not measured by this run.
NCU_DRAM_BYTES_PER_PAYLOAD_BYTE = {"restore_verify": 1.955, "restore": 1.955, "digest_verify": 1.008, "digest": 1.008,
                                   "kv_restore": 1.919, "capture": None}
NCU_TRAFFIC_SOURCE = ("profiles/stream_kernels_llama3-8b-shrink4_ncu_full.md, profiles/kv_stream_kernels_6GB_pool_ncu_full.md: "
                      "ncu dram__bytes of a small case of the same kernel, per payload byte, x this payload (not measured in this run)")
CONFIG_ORDER = ["tiny", "8b", "kv", "mixed", "host70b"]


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30, help="timed steps (a recovery restores once; long loops run power-capped)")
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["gms", "reference"], default="gms")
    ap.add_argument("--workload", choices=["8b", "mixed", "tiny", "kv", "host70b", "capture", "file"], default=None,
                    help="one workload only (default: the 8B headline plus all five configurations)")
    ap.add_argument("--unfused", action="store_true", help="8b/mixed/tiny: four calls per step instead of the two fused ones")
    ap.add_argument("--stage-buffers", type=int, default=3, help="device ring of the copy-engine-fed host restore")
    ap.add_argument("--stage-mib", type=int, default=64)
    ap.add_argument("--vmm", action="store_true", help="8b/mixed/tiny/capture/file: destinations from gms_service VMM slabs")
    ap.add_argument("--graph", action="store_true",
                    help="8b/mixed/tiny: capture the step into a CUDA graph once and time its replays (whole step only)")
    ap.add_argument("--no-l2-flush", action="store_true", help="mixed/tiny: leave L2 as the previous step left it")
    ap.add_argument("--file-dir", default="/dev/shm", help="file: where the snapshot file is written")
    ap.add_argument("--no-file", action="store_true", help="default run: leave the storage-fed entry out")
    ap.add_argument("--pipe-buffers", type=int, default=4)
    ap.add_argument("--pipe-mib", type=int, default=256)
    ap.add_argument("--pipe-readers", type=int, default=16)
    ap.add_argument("--direct-io", action="store_true", help="file: O_DIRECT reads where the file system takes them (cold files on fast storage)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=12.0, help="target CPU time of the headline's oracle sample")
    ap.add_argument("--cpu-seconds-other", type=float, default=4.0, help="the same for each of the other configurations")
    ap.add_argument("--host-gib", type=float, default=32.0, help="host70b: size of the pinned host image")
    ap.add_argument("--kv-gb", type=float, default=60.0, help="kv: size of the paged pool (a small pool is used for ncu captures)")
    ap.add_argument("--shrink", type=int, default=1, help="8b: divide the hidden sizes (a small manifest of the same structure, for ncu captures)")
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
        self.samples = []  # (t, sm_mhz, reasons_bitmask, mem_mhz, watts)
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
    """The step over a manifest workload (8b / mixed / tiny): digest + verify + restore + verify, as two fused
    calls (default) or four separate ones."""

    def __init__(self, name, torch, gms, W, dev, fused=True, vmm=False, shrink=1):
        self.torch, self.gms, self.W, self.dev, self.name, self.fused = torch, gms, W, dev, name, fused
        self.w = {"8b": lambda: W.llama3_8b_manifest(shrink=shrink), "mixed": W.mixed_manifest, "tiny": W.tiny_manifest}[name]()
        w = self.w
        self.image = torch.empty(w.image_bytes, dtype=torch.uint8, device=dev)
        W.fill_random_device(self.image, W.SEED_BASE + 0x100)
        self.vmm = vmm  # destinations carved from gms_service slabs
        self.svc = None
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
        gms.gms_manifest_build(self.entries[:1], w.image_bytes).close()  # first call on a device sets the launch shapes up
        torch.cuda.synchronize()  # the build synchronises the default stream: keep the fills above out of its time
        t0 = time.perf_counter()
        self.m = gms.gms_manifest_build(self.entries, w.image_bytes)
        self.build_ms = (time.perf_counter() - t0) * 1e3  # host: validation, work lists, upload of the tables
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
        n_dchunks = (nb + 7) // 8  # the digest-only kernel walks its own list of 8-block chunks (upper bound)
        self.bytes_digest = self.payload + 8 * nb + 32 * n_dchunks
        self.bytes_restore = 2 * self.payload + 8 * nb + 32 * self.n_chunks
        self.bytes_verify = 16 * nb
        self.set_fused(fused)
        self.launches_per_step = None
        self.graph = None
        # a working set that L2 (126 MB) could hold between steps is flushed out before every step
        self.l2_flush = torch.zeros(256 << 20, dtype=torch.uint8, device=dev) if self.payload < (512 << 20) else None

    def set_fused(self, fused: bool):
        """Two fused calls per step (digest + verify, restore + verify in one pass each) or the four separate ones."""
        nb = self.m.n_blocks
        self.fused = fused
        if fused:
            self.phase_names = ["digest_verify", "restore_verify"]
            self.phase_bytes = {"digest_verify": self.bytes_digest + 8 * nb, "restore_verify": self.bytes_restore + 8 * nb}
            self.dominant = "restore_verify"
        else:
            self.phase_names = ["digest", "verify", "restore", "verify2"]
            self.phase_bytes = {"digest": self.bytes_digest, "verify": self.bytes_verify, "restore": self.bytes_restore,
                                "verify2": self.bytes_verify}
            self.dominant = "restore"
        self.traffic = sum(self.phase_bytes.values())

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

    def step(self, marks=None):
        g, m = self.gms, self.m
        if self.graph is not None:
            if marks: marks[0].record()
            self.graph.replay()
            if marks:
                for e in marks[1:]: e.record()
            return
        if marks: marks[0].record()
        if self.fused:
            g.gms_digest_verify(m, self.bd, self.td, self.mm, self.cap, self.cnt)
            if marks: marks[1].record()
            g.gms_restore_verify(m, self.image, g.SRC_DEVICE, self.bd, self.td, self.mm, self.cap, self.cnt)
            if marks: marks[2].record()
            return
        g.gms_digest(m, self.bd, self.td)
        if marks: marks[1].record()
        g.gms_verify(m, self.bd, self.mm, self.cap, self.cnt)
        if marks: marks[2].record()
        g.gms_restore(m, self.image, g.SRC_DEVICE, self.bd, self.td)
        if marks: marks[3].record()
        g.gms_verify(m, self.bd, self.mm, self.cap, self.cnt)
        if marks: marks[4].record()

    def check(self) -> bool:
        """Parity flag of the run: the last verify found nothing and no bounded wait expired."""
        self.torch.cuda.synchronize()
        return int(self.cnt.item()) == 0 and self.gms.gms_last_device_status(self.m) == 0

    def step_text(self):
        return ("gms_digest_verify + gms_restore_verify(device image)" if self.fused
                else "gms_digest + gms_verify + gms_restore(device image) + gms_verify")

    def config(self):
        return {"workload": f"{self.w.name}: {len(self.w.rows)} tensors, {self.payload} B payload, "
                            f"{self.m.n_blocks} digest blocks, {self.n_chunks} chunks",
                "step": self.step_text(),
                "destinations": "gms_service VMM slabs (2 GiB, first fit)" if self.vmm else "carved from one cudaMalloc slab",
                "l2": "inputs larger than L2 (no flush)" if self.payload >= (512 << 20) else
                      ("L2 flushed before every step (256 MiB read+write, outside the phase events); ms_per_step = sum of phases"
                       if self.l2_flush is not None else "working set near L2 size; not flushed"),
                "payload_bytes": self.payload}

    def kernel_text(self):
        return (f"gms_stream_kernel ({self.dominant}; duration = the call's events: one-block prologue + streaming kernel"
                + (" + the one small emit kernel of the fused verify)" if self.fused else ")"))

    def close(self):
        self.m.close()
        if self.svc is not None:
            self.svc.close()


class CaptureBench(ManifestBench):
    """gms_capture of the 8B manifest (allocations -> packed device image, fused digest) + gms_verify."""

    def __init__(self, torch, gms, W, dev, vmm=False):
        super().__init__("8b", torch, gms, W, dev, fused=False, vmm=vmm)
        self.phase_names = ["capture", "verify"]
        self.phase_bytes = {"capture": self.bytes_restore, "verify": self.bytes_verify}
        self.dominant = "capture"
        self.traffic = self.bytes_restore + self.bytes_verify

    def step(self, marks=None):
        g, m = self.gms, self.m
        if marks: marks[0].record()
        g.gms_capture(m, self.image, g.SRC_DEVICE, self.bd, self.td)
        if marks: marks[1].record()
        g.gms_verify(m, self.bd, self.mm, self.cap, self.cnt)
        if marks: marks[2].record()

    def step_text(self):
        return "gms_capture(device image) + gms_verify"


class KvBench:
    """gms_kv_restore of a seeded 10% of a paged KV pool, gms_kv_digest of the same blocks in place, gms_kv_verify."""

    def __init__(self, torch, gms, W, dev, pool_bytes=60e9):
        self.torch, self.gms, self.name = torch, gms, "kv"
        k = self.k = W.kv_pool_workload(pool_bytes=pool_bytes)
        self.pool = torch.empty(k.pool_bytes, dtype=torch.uint8, device=dev)
        W.fill_random_device(self.pool, W.SEED_BASE + 0x200)
        self.image = torch.empty(k.image_bytes, dtype=torch.uint8, device=dev)
        W.fill_random_device(self.image, W.SEED_BASE + 0x201)
        self.ids = torch.from_numpy(k.ids).to(dev)
        kk = k.block_bytes // 4096
        n_slots = len(k.ids) * k.n_planes * kk
        self.bd = torch.zeros(n_slots, dtype=torch.int64, device=dev)
        self.kd = torch.zeros(len(k.ids), dtype=torch.int64, device=dev)
        self.st = torch.zeros(4, dtype=torch.int64, device=dev)
        self.desc = gms.KvPool(base=self.pool.data_ptr(), plane_stride=k.plane_stride, block_stride=k.block_stride,
                               n_planes=k.n_planes, n_blocks=k.n_blocks, block_bytes=k.block_bytes)
        self.payload = k.payload_bytes
        self.bytes_restore = 2 * self.payload + 8 * n_slots
        self.bytes_digest = self.payload + 8 * n_slots
        self.bytes_verify = 16 * n_slots
        self.phase_names = ["kv_restore", "kv_digest", "kv_verify"]
        self.phase_bytes = {"kv_restore": self.bytes_restore, "kv_digest": self.bytes_digest, "kv_verify": self.bytes_verify}
        self.traffic = sum(self.phase_bytes.values())
        self.dominant = "kv_restore"
        # digests of the restore, against which the in-place digests are verified
        self.bd_restore = torch.zeros_like(self.bd)
        self.mm = torch.zeros(2 * 64, dtype=torch.int64, device=dev)  # 64 records of 16 bytes
        self.cnt = torch.zeros(1, dtype=torch.int64, device=dev)
        self.scratch = torch.zeros(gms.kv_verify_scratch_words(n_slots), dtype=torch.int32, device=dev)
        self.l2_flush = None

    def step(self, marks=None):
        g, k = self.gms, self.k
        if marks: marks[0].record()
        g.gms_kv_restore(self.desc, self.image, k.img_plane_stride, k.img_slot_stride, g.SRC_DEVICE, self.ids, len(k.ids),
                         self.bd_restore, self.kd, self.st)
        if marks: marks[1].record()
        g.gms_kv_digest(self.desc, self.ids, len(k.ids), self.bd, self.kd, self.st)
        if marks: marks[2].record()
        g.gms_kv_verify(self.desc, self.ids, len(k.ids), self.bd, self.bd_restore, self.mm, 64, self.cnt, self.scratch)
        if marks: marks[3].record()

    def check(self) -> bool:
        self.torch.cuda.synchronize()
        return self.st[:2].tolist() == [0, 0] and int(self.cnt.item()) == 0

    def step_text(self):
        return "gms_kv_restore(device image) + gms_kv_digest(the same blocks in place) + gms_kv_verify"

    def config(self):
        k = self.k
        return {"workload": f"{k.name}: pool {k.pool_bytes} B, {len(k.ids)} of {k.n_blocks} blocks selected, {self.payload} B moved",
                "step": self.step_text(), "l2": "inputs larger than L2 (no flush)", "payload_bytes": self.payload}

    def kernel_text(self):
        return "gms_kv_stream_kernel (kv_restore; duration = the call's events, incl. its one-block prologue)"

    def close(self):
        pass


def event_list(torch, n):
    return [torch.cuda.Event(enable_timing=True) for _ in range(n)]


def timed_steps(torch, bench, steps, dist=None):
    """Times `steps` steps with CUDA events on the current stream.

    Returns (total ms, {phase: {"mean", "median", "best"}} in ms, (t0, t1) host times of the timed region).
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
        bench.step(marks[i])
    e1.record()
    torch.cuda.synchronize()
    t1 = time.perf_counter()
    if dist is not None and dist.is_initialized():
        dist.barrier()
        torch.cuda.synchronize()
    total = e0.elapsed_time(e1)
    stats = {}
    for p, name in enumerate(bench.phase_names):
        ts = [marks[i][p].elapsed_time(marks[i][p + 1]) for i in range(steps)]
        stats[name] = {"mean": statistics.fmean(ts), "median": statistics.median(ts), "best": min(ts)}
    if flush is not None:
        total = sum(s["mean"] for s in stats.values()) * steps
    return total, stats, (t0, t1)


def measure(torch, gms, bench, steps, warmup, index, dist=None, dev=None, graph=False):
    """Warm-up, timed steps with the clocks sampled during them, and the entry that describes the run."""
    peak, peak_kind = measured_peak()
    for _ in range(max(warmup, 3)):
        bench.step()
    ok = bench.check()
    if graph:
        bench.use_graph()
        for _ in range(3):
            bench.step()
        ok = ok and bench.check()
    sampler = ClockSampler(index)
    launches0 = gms.gms_kernel_launches()
    sampler.start()
    total_ms, stats, (t0, t1) = timed_steps(torch, bench, steps, dist)
    sampler.stop()
    launches = gms.gms_kernel_launches() - launches0
    if graph:  # replays do not pass through the library's launch counter
        launches = bench.launches_per_step * steps
    ok = ok and bench.check()
    max_ms, sum_traffic = reduce_over_ranks(total_ms, float(bench.traffic) * steps, dist, dev)
    phases = {}
    for name, s in stats.items():
        b = bench.phase_bytes[name]
        gbs = b / s["median"] / 1e6
        phases[name] = {"mean_ms": s["mean"], "median_ms": s["median"], "best_ms": s["best"], "bytes": b, "gbs": gbs,
                        "frac_of_measured": gbs / peak, "frac_of_8TBps": gbs / DATASHEET_HBM_GBS}
    if graph:  # one event pair around each replay: the whole step's bytes over the whole step's time
        achieved = bench.traffic / (total_ms / steps) / 1e6
        roofline = {"kernel": "whole step replayed from a CUDA graph", "bound": "hbm", "achieved": achieved, "peak": peak,
                    "unit": "GB/s", "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                    "frac_of_datasheet_8TBps": achieved / DATASHEET_HBM_GBS, "algorithmic_bytes_per_launch": bench.traffic,
                    "traffic": None}
        phases = {"step": {"mean_ms": total_ms / steps}}
    else:
        dom = bench.dominant
        achieved = bench.phase_bytes[dom] / stats[dom]["mean"] / 1e6
        ratio = NCU_DRAM_BYTES_PER_PAYLOAD_BYTE.get(dom)
        roofline = {"kernel": bench.kernel_text(), "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                    "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "frac_of_datasheet_8TBps": achieved / DATASHEET_HBM_GBS,
                    "achieved_median": bench.phase_bytes[dom] / stats[dom]["median"] / 1e6,
                    "frac_median": bench.phase_bytes[dom] / stats[dom]["median"] / 1e6 / peak,
                    "duration_ms": {"mean": stats[dom]["mean"], "median": stats[dom]["median"], "best": stats[dom]["best"]},
                    "algorithmic_bytes_per_launch": bench.phase_bytes[dom], "traffic": (ratio * bench.payload) if ratio else None,
                    "traffic_source": NCU_TRAFFIC_SOURCE if ratio else None}
    return {
        "workload": bench.config()["workload"], "step": bench.step_text(), "steps": steps, "warmup": max(warmup, 3),
        "ms_per_step": max_ms / steps, "value": sum_traffic / max_ms / 1e6, "unit": UNIT, "bytes_per_step": bench.traffic,
        "payload_bytes": bench.payload, "phases": phases, "roofline": roofline, "clocks": sampler.summary(t0, t1),
        "gpu_launches": int(launches), "parity_ok": bool(ok), "l2": bench.config()["l2"],
        "manifest_build_ms": getattr(bench, "build_ms", None),
    }


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


def make_oracle_sample(oracle, w, sample_bytes, image_fetch):
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


def sized_oracle_sample(oracle, w, fetch, seconds, calibrate_bytes=32 << 20, max_bytes=8 << 30):
    """A prefix sample of the workload sized for about `seconds` of one oracle step (calibrated on a small prefix)."""
    rec, image, slab, expected, used, _ = make_oracle_sample(oracle, w, calibrate_bytes, fetch)
    t = time.perf_counter()
    oracle_step(oracle, rec, image, slab, expected)
    per_byte = (time.perf_counter() - t) / max(used, 1)
    target = int(min(max(seconds / per_byte, calibrate_bytes), max_bytes))
    return make_oracle_sample(oracle, w, target, fetch)


def cpu_baseline_manifest(w, fetch, seconds, all_cores=False, what="manifest"):
    """Times the oracle, as it stands, on a bounded prefix sample of the same workload (1 thread)."""
    from oracle import gms_oracle as oracle

    rec, image, slab, expected, used, n = sized_oracle_sample(oracle, w, fetch, seconds)
    t = time.perf_counter()
    bad = oracle_step(oracle, rec, image, slab, expected)
    dt = time.perf_counter() - t
    assert bad == 0
    nb = int(sum((int(r[3]) + 4095) // 4096 for r in rec))
    traffic = 3 * used + 16 * nb + 2 * 16 * nb
    whole = n == len(w.rows)
    out = {"value": traffic / dt / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle", "seconds": dt,
           "sample": (f"all {n} tensors" if whole else f"first {n} of {len(w.rows)} tensors") +
                     f" of the {what} ({used} B payload), step = digest+verify+restore+verify, 1 of {os.cpu_count()} host cores"}
    if not all_cores:
        return out
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


def oracle_kv_step(oracle, k, planes, pool, image):
    """kv_restore + kv_digest + kv_verify on the first `planes` planes.  Returns (mismatch count, bytes moved, slots)."""
    rc, bd, kd, skipped = oracle.kv_restore(pool, k.plane_stride, k.block_stride, planes, k.n_blocks, k.block_bytes, image,
                                            k.img_plane_stride, k.img_slot_stride, k.ids)
    rc2, bd2, kd2, _ = oracle.kv_digest(pool, k.plane_stride, k.block_stride, planes, k.n_blocks, k.block_bytes, k.ids)
    count, _ = oracle.kv_verify(planes, k.n_blocks, k.block_bytes, k.ids, bd2, bd, 64)
    assert rc == 0 and rc2 == 0 and skipped == 0 and (kd2 == kd).all()
    return count, planes * len(k.ids) * k.block_bytes, bd.size


def cpu_baseline_kv(k, image_fetch, planes=16):
    """The oracle's kv_restore + kv_digest + kv_verify (1 thread) on the first `planes` planes of the same pool
    shape, image and id list.  image_fetch(nbytes) returns the first nbytes of the packed image as numpy."""
    import numpy as np

    from oracle import gms_oracle as oracle

    planes = min(planes, k.n_planes)
    image = image_fetch(planes * k.img_plane_stride)
    pool = np.empty(planes * k.plane_stride, dtype=np.uint8)  # only the selected blocks are ever touched
    # touch every page the step will write, so that the timing below is the oracle's work and not first-touch page faults
    ids = k.ids[(k.ids >= 0) & (k.ids < k.n_blocks)].astype(np.int64)
    pages = (np.arange(planes, dtype=np.int64)[:, None, None] * k.plane_stride + ids[None, :, None] * k.block_stride
             + np.arange(0, k.block_bytes, 4096, dtype=np.int64)[None, None, :])
    pool[pages.ravel()] = 0
    t = time.perf_counter()
    count, moved, slots = oracle_kv_step(oracle, k, planes, pool, image)
    dt = time.perf_counter() - t
    assert count == 0
    out = {"value": (3 * moved + 32 * slots) / dt / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle", "seconds": dt,
           "sample": f"kv_restore + kv_digest + kv_verify on the first {planes} of {k.n_planes} planes of the same pool, image and "
                     f"id list ({moved} B moved), 1 of {os.cpu_count()} host cores"}
    # the same oracle calls on all host cores: one plane per thread (the oracle is untouched; ctypes releases the GIL)
    import concurrent.futures as cf
    import dataclasses

    one = dataclasses.replace(k)  # same shape and id list; each thread is handed one plane of pool and image

    def plane(p):
        return oracle_kv_step(oracle, one, 1, pool[p * k.plane_stride:(p + 1) * k.plane_stride],
                              image[p * k.img_plane_stride:(p + 1) * k.img_plane_stride])[0]

    with cf.ThreadPoolExecutor(min(planes, os.cpu_count() or 1)) as ex:
        t = time.perf_counter()
        bad = sum(ex.map(plane, range(planes)))
        dt_all = time.perf_counter() - t
    assert bad == 0
    out["all_cores"] = {"value": (3 * moved + 32 * slots) / dt_all / 1e9, "unit": UNIT, "cores": min(planes, os.cpu_count() or 1),
                        "seconds": dt_all}
    return out


def cpu_baseline_host(w, arr, seconds):
    """The oracle's restore + verify (1 thread) on a prefix of the host-image manifest, reading the pinned image itself."""
    from oracle import gms_oracle as oracle

    fetch = lambda lo, hi: arr[lo:hi]
    rec, image, slab, expected, used, n = sized_oracle_sample(oracle, w, fetch, seconds * 2.0)  # this step is half the 4-call one
    t = time.perf_counter()
    _, bd, _ = oracle.restore(rec, image, slab)
    bad, _ = oracle.verify(rec, bd, expected, 64)
    dt = time.perf_counter() - t
    assert bad == 0
    out = {"value": used / dt / 1e9, "unit": "GB/s of payload", "cores": 1, "kind": "oracle", "seconds": dt,
           "sample": f"first {n} of {len(w.rows)} tensors of the host-image manifest ({used} B payload), step = restore+verify, "
                     f"1 of {os.cpu_count()} host cores"}
    # all host cores: the sample's tensors dealt out to one thread each (largest first), same oracle calls
    import concurrent.futures as cf

    cores = os.cpu_count() or 1
    order = sorted(range(len(rec)), key=lambda i: -int(rec[i]["nbytes"]))
    loads, groups = [0] * cores, [[] for _ in range(cores)]
    for i in order:
        j = loads.index(min(loads))
        groups[j].append(i)
        loads[j] += int(rec[i]["nbytes"])
    shards = []
    for g in groups:
        if g:
            sub = rec[sorted(g)]
            _, exp_sub, _ = oracle.digest(sub, slab)
            shards.append((sub, exp_sub))

    def shard_step(sh):
        _, b, _ = oracle.restore(sh[0], image, slab)
        return oracle.verify(sh[0], b, sh[1], 64)[0]

    with cf.ThreadPoolExecutor(len(shards)) as ex:
        t = time.perf_counter()
        bad = sum(ex.map(shard_step, shards))
        dt_all = time.perf_counter() - t
    assert bad == 0
    out["all_cores"] = {"value": used / dt_all / 1e9, "unit": "GB/s of payload", "cores": len(shards), "seconds": dt_all}
    return out


def reference_arm(args):
    """`--impl reference`: the oracle on this host's cores, same metric, bounded sample per step."""
    rank, _, world = dist_env()
    if rank != 0:
        return
    import numpy as np

    from oracle import gms_oracle as oracle
    from paper_2609_25451_b200 import workloads as W

    workload = args.workload or "8b"
    per_step_s = min(3.0, 150.0 / max(args.steps + args.warmup, 1))
    rng_image = {}

    def fetch(lo, hi):  # synthetic bytes generated on the host for the sampled range only
        key = (lo, hi)
        if key not in rng_image:
            rng_image[key] = W.random_bytes_host(hi - lo, seed=(W.SEED_BASE + lo) & 0x7FFFFFFF)
        return rng_image[key]

    if workload == "kv":
        k = W.kv_pool_workload(pool_bytes=args.kv_gb * 1e9)
        # planes sized for the per-step budget (one plane moves 94 MB; the oracle does about 0.5 GB/s of this step)
        planes = int(max(1, min(k.n_planes, per_step_s * 0.5e9 / (3 * len(k.ids) * k.block_bytes))))
        image = W.random_bytes_host(planes * k.img_plane_stride, seed=W.SEED_BASE + 0x201)
        pool = np.empty(planes * k.plane_stride, dtype=np.uint8)
        run = lambda: oracle_kv_step(oracle, k, planes, pool, image)
        count, moved, slots = run()
        step_bytes = 3 * moved + 32 * slots
        name, used = k.name, moved
        sample = f"each step: kv_restore + kv_digest + kv_verify on the first {planes} of {k.n_planes} planes ({moved} B moved), 1 thread"
        check = lambda r: r[0] == 0
    else:
        host_step = workload == "host70b"
        w = {"8b": W.llama3_8b_manifest, "mixed": W.mixed_manifest, "tiny": W.tiny_manifest, "capture": W.llama3_8b_manifest,
             "file": W.llama3_8b_manifest,
             "host70b": lambda: W.llama3_70b_tp8_shard_manifest(image_bytes=int(args.host_gib * (1 << 30)) // 16 * 16)}[workload]()
        rec, image, slab, expected, used, n = sized_oracle_sample(oracle, w, fetch, per_step_s * (2.0 if host_step else 1.0),
                                                                  calibrate_bytes=16 << 20, max_bytes=4 << 30)
        nb = int(sum((int(r[3]) + 4095) // 4096 for r in rec))
        if host_step:  # the host-sourced step: restore + verify
            def run():
                _, bd, _ = oracle.restore(rec, image, slab)
                return oracle.verify(rec, bd, expected, 64)[0]
            step_bytes = 2 * used + 24 * nb
            sample = f"each step: first {n} tensors of {w.name} ({used} B payload), restore+verify, 1 thread"
        else:
            run = lambda: oracle_step(oracle, rec, image, slab, expected)
            step_bytes = 3 * used + 48 * nb
            sample = f"each step: first {n} tensors of {w.name} ({used} B payload), digest+verify+restore+verify, 1 thread"
        name = w.name
        check = lambda r: r == 0
    for _ in range(args.warmup):
        run()
    t = time.perf_counter()
    for _ in range(args.steps):
        assert check(run())
    dt = time.perf_counter() - t
    value = step_bytes * args.steps / dt / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / max(args.steps, 1) * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u64", "data": "synthetic",
        "config": {"workload": f"{name} (bounded sample per step)", "payload_bytes": used},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------- host-sourced legs
def host_image_of(torch, gms, dev_image):
    """Pinned, device-mapped host copy of a device image.  Returns (host_ptr, device_view, cpu tensor)."""
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


def e2e_leg(args, torch, gms, bench, dist, dev):
    """The step with the snapshot image in pinned HOST memory: it crosses the link inside gms_restore_staged (copy
    engine -> device ring -> restore kernel) and the verdict comes back to pinned host memory, every step."""
    hptr, dview, cpu = host_image_of(torch, gms, bench.image)
    h2d_gbs = h2d_yardstick(torch, cpu, bench.image)
    pin_cnt = torch.zeros(1, dtype=torch.int64).pin_memory()
    pin_td = torch.zeros(bench.td.numel(), dtype=torch.int64).pin_memory()
    stage = gms.gms_stage_create(args.stage_buffers, args.stage_mib << 20)

    class E2E:
        phase_names = ["digest_verify", "restore", "verify", "readback"]
        l2_flush = None

        @staticmethod
        def step(marks=None):
            g, m = gms, bench.m
            if marks: marks[0].record()
            g.gms_digest_verify(m, bench.bd, bench.td, bench.mm, bench.cap, bench.cnt)
            if marks: marks[1].record()
            g.gms_restore_staged(m, stage, hptr, bench.bd, bench.td)
            if marks: marks[2].record()
            g.gms_verify(m, bench.bd, bench.mm, bench.cap, bench.cnt)
            if marks: marks[3].record()
            pin_cnt.copy_(bench.cnt, non_blocking=True)
            pin_td.copy_(bench.td, non_blocking=True)
            if marks: marks[4].record()

    steps = max(args.e2e_steps, 1)
    E2E.step()
    torch.cuda.synchronize()
    e_ms, e_stats, _ = timed_steps(torch, E2E, steps, dist)
    ok = int(pin_cnt.item()) == 0
    e_max, e_traffic = reduce_over_ranks(e_ms, float(bench.traffic) * steps, dist, dev)
    # for comparison: the same restore with kernel-issued reads of the mapped image (no copy engine)
    ma, mb = event_list(torch, 2)
    ma.record()
    gms.gms_restore(bench.m, dview, gms.SRC_HOST_MAPPED, bench.bd, bench.td)
    mb.record()
    torch.cuda.synchronize()
    mapped_gbs = bench.payload / ma.elapsed_time(mb) / 1e6
    r_gbs = bench.payload / e_stats["restore"]["mean"] / 1e6
    out = {
        "value": e_traffic / e_max / 1e6, "unit": UNIT, "h2d_bytes_per_step": bench.payload,
        "d2h_bytes_per_step": 8 + 8 * bench.td.numel(), "steps": steps, "ms_per_step": e_max / steps,
        "payload_gbs": bench.payload * (e_traffic / float(bench.traffic) / steps) / (e_max / steps) / 1e6,
        "value_note": "value = the step's algorithmic HBM bytes (3 x payload) per second, as in the device-timed line; "
                      "payload_gbs = snapshot payload per second of the same end-to-end step, which the host link bounds",
        "call": f"gms_digest_verify + gms_restore_staged ({args.stage_buffers} x {args.stage_mib} MiB device ring) + gms_verify + D2H of the verdict",
        "host_restore_gbs": r_gbs, "h2d_memcpy_gbs": h2d_gbs, "host_restore_frac_of_memcpy": r_gbs / h2d_gbs,
        "host_mapped_restore_gbs": mapped_gbs, "host_mapped_frac_of_memcpy": mapped_gbs / h2d_gbs, "parity_ok": bool(ok),
    }
    torch.cuda.synchronize()
    stage.close()
    gms.gms_host_image_free(hptr)
    return out


def kv_host_legs(torch, gms, bench, reps=3):
    """The KV subset moved across the host link (Section 6: committed KV blocks kept in host memory): gms_kv_capture of
    the selected blocks into a pinned, mapped host image and gms_kv_restore back from it, against plain cudaMemcpyAsync
    of the same number of bytes in each direction through the same pinned buffer."""
    k = bench.k
    hptr, dview, arr = gms.gms_host_image_alloc(k.image_bytes)
    try:
        cpu = torch.from_numpy(arr)
        n_sel = len(k.ids)

        def best_of(fn, n):
            ts = []
            for _ in range(n):
                a, b = event_list(torch, 2)
                a.record()
                fn()
                b.record()
                torch.cuda.synchronize()
                ts.append(a.elapsed_time(b))
            return min(ts)

        d2h = k.image_bytes / best_of(lambda: cpu.copy_(bench.image, non_blocking=True), reps + 1) / 1e6
        h2d = k.image_bytes / best_of(lambda: bench.image.copy_(cpu, non_blocking=True), reps + 1) / 1e6
        cap_ms = best_of(lambda: gms.gms_kv_capture(bench.desc, dview, k.img_plane_stride, k.img_slot_stride, gms.SRC_HOST_MAPPED,
                                                    bench.ids, n_sel, bench.bd_restore, bench.kd, bench.st), reps)
        ok = bench.st[:2].tolist() == [0, 0]
        res_ms = best_of(lambda: gms.gms_kv_restore(bench.desc, dview, k.img_plane_stride, k.img_slot_stride, gms.SRC_HOST_MAPPED,
                                                    bench.ids, n_sel, bench.bd, bench.kd, bench.st), reps)
        # what was captured from the pool is what is put back: the two calls must report the same digests
        ok = ok and bench.st[:2].tolist() == [0, 0] and bool(torch.equal(bench.bd, bench.bd_restore))
        cap, res = bench.payload / cap_ms / 1e6, bench.payload / res_ms / 1e6
        return {"kv_capture_to_host": {"ms": cap_ms, "achieved": cap, "peak": d2h, "frac": cap / d2h, "unit": "GB/s"},
                "kv_restore_from_host": {"ms": res_ms, "achieved": res, "peak": h2d, "frac": res / h2d, "unit": "GB/s"},
                "bound": "host_link", "peak_kind": "cudaMemcpyAsync of the packed image through the same pinned buffer, same run",
                "bytes": bench.payload, "parity_ok": ok}
    finally:
        torch.cuda.synchronize()
        gms.gms_host_image_free(hptr)


def capture_to_host_leg(torch, gms, bench, reps=3):
    """gms_capture of the same allocations into a pinned, mapped HOST image (the snapshot direction: device state
    staged into host memory), against a plain cudaMemcpyAsync device->host of the same bytes into the same buffer."""
    hptr, dview, arr = gms.gms_host_image_alloc(bench.w.image_bytes)
    try:
        cpu = torch.from_numpy(arr)
        best_copy = None
        for _ in range(reps + 1):
            a, b = event_list(torch, 2)
            a.record()
            cpu.copy_(bench.image, non_blocking=True)
            b.record()
            torch.cuda.synchronize()
            best_copy = a.elapsed_time(b) if best_copy is None else min(best_copy, a.elapsed_time(b))
        d2h_gbs = bench.w.image_bytes / best_copy / 1e6
        times = []
        for _ in range(reps):
            a, b = event_list(torch, 2)
            a.record()
            gms.gms_capture(bench.m, dview, gms.SRC_HOST_MAPPED, bench.bd, bench.td)
            b.record()
            torch.cuda.synchronize()
            times.append(a.elapsed_time(b))
        gms.gms_verify(bench.m, bench.bd, bench.mm, bench.cap, bench.cnt)
        ok = bench.check()
        gbs = bench.payload / min(times) / 1e6
        return {"call": "gms_capture(host-mapped image): kernel-issued bulk stores across the host link", "ms": min(times),
                "achieved": gbs, "peak": d2h_gbs, "unit": "GB/s", "frac": gbs / d2h_gbs, "bound": "host_link",
                "peak_kind": "cudaMemcpyAsync D2H of the image into the same pinned buffer, same run, best of 4",
                "d2h_bytes": bench.payload, "parity_ok": bool(ok)}
    finally:
        torch.cuda.synchronize()
        gms.gms_host_image_free(hptr)


def run_host70b(args, torch, gms, W, dev, index, want_cpu=True, cpu_seconds=4.0):
    """Host-sourced restore of a Llama-3-70B TP8 shard manifest from a pinned, mapped host image,
    against a plain cudaMemcpyAsync of the same bytes from the same allocation.  Returns the config entry."""
    import numpy as np

    image_bytes = int(args.host_gib * (1 << 30)) // 16 * 16
    w = W.llama3_70b_tp8_shard_manifest(image_bytes=image_bytes)
    hptr, dview, arr = gms.gms_host_image_alloc(w.image_bytes)
    try:
        cpu = torch.from_numpy(arr)
        scratch = torch.empty(1 << 30, dtype=torch.uint8, device=dev)
        for i, a in enumerate(range(0, w.image_bytes, 1 << 30)):  # random bits made on the GPU, copied to the host image
            n = min(1 << 30, w.image_bytes - a)
            W.fill_random_device(scratch[:n], W.SEED_BASE + 0x500 + i)
            cpu[a:a + n].copy_(scratch[:n])
        del scratch
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
        steps = max(1, min(args.steps, 3))
        sampler = ClockSampler(index)
        launches0 = gms.gms_kernel_launches()
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
        ok = int(cnt.item()) == 0 and gms.gms_last_device_status(m) == 0
        mapped = [ev[i][0].elapsed_time(ev[i][1]) for i in range(steps)]
        tot = statistics.fmean(ev[i][0].elapsed_time(ev[i][2]) for i in range(steps))
        # the copy-engine-fed variant of the same restore (device ring, windows ordered by stream events)
        stage = gms.gms_stage_create(args.stage_buffers, args.stage_mib << 20)
        gms.gms_restore_staged(m, stage, hptr, bd, td)
        torch.cuda.synchronize()
        ev = [event_list(torch, 3) for _ in range(steps)]
        for i in range(steps):
            ev[i][0].record()
            gms.gms_restore_staged(m, stage, hptr, bd, td)
            ev[i][1].record()
            gms.gms_verify(m, bd, mm, 64, cnt)
            ev[i][2].record()
        torch.cuda.synchronize()
        t1 = time.perf_counter()
        sampler.stop()
        launches = gms.gms_kernel_launches() - launches0
        ok = ok and int(cnt.item()) == 0 and gms.gms_last_device_status(m) == 0
        staged = [ev[i][0].elapsed_time(ev[i][1]) for i in range(steps)]
        s_tot = statistics.fmean(ev[i][0].elapsed_time(ev[i][2]) for i in range(steps))

        def phase(ts):
            gbs = w.payload_bytes / statistics.median(ts) / 1e6
            return {"mean_ms": statistics.fmean(ts), "median_ms": statistics.median(ts), "best_ms": min(ts), "bytes": w.payload_bytes,
                    "gbs": gbs, "frac_of_memcpy": gbs / h2d}

        phases = {"restore_mapped": phase(mapped), "restore_staged": phase(staged)}
        s_gbs = w.payload_bytes / min(staged) / 1e6
        m_gbs = w.payload_bytes / min(mapped) / 1e6
        shard = 17640718336  # one 70B TP8 shard; the image holds about 1.95 of them
        entry = {
            "workload": f"{w.name}: {len(w.rows)} tensors, {w.payload_bytes} B payload in a {w.image_bytes} B pinned mapped host image",
            "step": f"gms_restore_staged ({args.stage_buffers} x {args.stage_mib} MiB device ring, copy engine on the link) + gms_verify; "
                    "also timed: gms_restore(host-mapped image, kernel-issued reads) + gms_verify",
            "steps": steps, "warmup": 1, "ms_per_step": s_tot, "ms_per_step_mapped": tot, "value": w.payload_bytes / s_tot / 1e6,
            "unit": "GB/s of payload", "payload_bytes": w.payload_bytes, "bytes_per_step": w.payload_bytes, "phases": phases,
            "roofline": {"kernel": "gms_restore_staged: cudaMemcpyAsync windows on the copy engine -> device ring -> gms_stream_kernel (restore)",
                         "bound": "host_link", "achieved": s_gbs, "peak": h2d, "unit": "GB/s", "frac": s_gbs / h2d,
                         "peak_kind": "cudaMemcpyAsync H2D of the whole payload from the same pinned allocation, same run, best of 5",
                         "mapped_achieved": m_gbs, "mapped_frac": m_gbs / h2d, "h2d_memcpy_1gib_gbs": h2d_1gib, "traffic": None},
            "one_shard_restore_s": {"mapped": shard / m_gbs / 1e9, "staged": shard / s_gbs / 1e9, "memcpy_h2d": shard / h2d / 1e9},
            "clocks": sampler.summary(t0, t1), "gpu_launches": int(launches), "parity_ok": bool(ok),
            "l2": "inputs larger than L2 (no flush)",
        }
        if want_cpu:
            entry["cpu_baseline"] = cpu_baseline_host(w, arr, cpu_seconds)
        torch.cuda.synchronize()
        stage.close()
        m.close()
        return entry
    finally:
        torch.cuda.synchronize()
        gms.gms_host_image_free(hptr)


def run_file(args, torch, gms, W, dev, index, want_cpu=True, steps_cap=5):
    """Storage-fed restore of the 8B manifest: file -> ring of pinned buffers -> device (gms_restore_fd),
    against (a) the same reader pool filling one pinned buffer with nothing consuming it and (b) the host link."""
    import concurrent.futures as cf

    import numpy as np

    bench = ManifestBench("8b", torch, gms, W, dev, fused=False, vmm=args.vmm)
    w = bench.w
    path = os.path.join(args.file_dir, f"gms_bench_image_{os.getpid()}.bin")
    n_buf, buf_bytes, n_readers = args.pipe_buffers, args.pipe_mib << 20, args.pipe_readers
    fs_type = "unknown"
    try:
        with open("/proc/mounts") as f:
            best = ""
            for ln in f:
                parts = ln.split()
                if len(parts) >= 3 and os.path.abspath(args.file_dir).startswith(parts[1]) and len(parts[1]) >= len(best):
                    best, fs_type = parts[1], parts[2]
    except OSError:
        pass
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
        # (b) link yardstick: plain cudaMemcpyAsync of one pinned buffer's worth
        link_gbs = h2d_yardstick(torch, torch.from_numpy(arr), bench.image[:buf_bytes], reps=5)
        gms.gms_host_image_free(hptr)
        pipe = gms.gms_pipe_create(n_buf, buf_bytes, n_readers)
        gms.gms_pipe_direct_io(pipe, args.direct_io)
        gms.gms_restore_fd(bench.m, pipe, fd, 0, bench.bd, bench.td)
        steps = max(1, min(args.steps, steps_cap))
        sampler = ClockSampler(index)
        launches0 = gms.gms_kernel_launches()
        sampler.start()
        t0 = time.perf_counter()
        stats = [gms.gms_restore_fd(bench.m, pipe, fd, 0, bench.bd, bench.td) for _ in range(steps)]
        t1 = time.perf_counter()
        sampler.stop()
        launches = gms.gms_kernel_launches() - launches0
        gms.gms_verify(bench.m, bench.bd, bench.mm, bench.cap, bench.cnt)
        ok = bench.check()
        best = min(s["total_seconds"] for s in stats)
        gbs = w.payload_bytes / best / 1e9
        bound = min(read_gbs, link_gbs)
        line = {
            "metric": "file-sourced restore+digest GB/s", "value": gbs, "unit": UNIT, "n_gpus": 1, "steps": steps, "warmup": 1,
            "ms_per_step": best * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u64",
            "data": "synthetic",
            "config": {"workload": f"{w.name}: {w.payload_bytes} B read from {args.file_dir} ({fs_type}) through {n_buf} x {args.pipe_mib} MiB "
                                   f"pinned buffers, {n_readers} reader threads", "step": "gms_restore_fd (wall clock, synchronous call)",
                       "l2": "inputs larger than L2 (no flush)", "file_system": fs_type},
            "roofline": {"bound": "storage_read" if read_gbs < link_gbs else "host_link", "achieved": gbs, "peak": bound, "unit": "GB/s",
                         "frac": gbs / bound, "reader_yardstick_gbs": read_gbs, "link_yardstick_gbs": link_gbs,
                         "peak_kind": "min(same file, same reader threads and slicing, into one pinned buffer with no consumer; "
                                      "plain cudaMemcpyAsync H2D of one pinned buffer)", "traffic": None},
            "pipe_stats_best": min(stats, key=lambda s: s["total_seconds"]),
            "clocks": sampler.summary(t0, t1), "gpu_launches": int(launches), "parity_ok": bool(ok),
        }
        if want_cpu:
            fetch = lambda lo, hi: bench.image[lo:hi].cpu().numpy()
            line["cpu_baseline"] = cpu_baseline_manifest(w, fetch, args.cpu_seconds_other, what="manifest (image in host memory)")
        os.close(fd)
        fd = -1
        os.remove(path)
        # ---- the way back: the restored allocations gathered into a new file (gms_capture_fd), against (a) the same
        # writer threads emptying one pinned buffer into the file with no GPU work and (b) the link, device to host
        with open(path, "wb") as f:
            f.truncate(w.image_bytes)
        wfd = os.open(path, os.O_WRONLY)
        hptr, _, arr = gms.gms_host_image_alloc(buf_bytes)
        mv = memoryview(arr)

        def write_all():
            with cf.ThreadPoolExecutor(n_readers) as ex:
                for lo in range(0, w.image_bytes, buf_bytes):
                    n = min(buf_bytes, w.image_bytes - lo)
                    futs = [ex.submit(os.pwritev, wfd, [mv[o:min(o + slice_b, n)]], lo + o) for o in range(0, n, slice_b)]
                    for fu in futs:
                        fu.result()

        write_all()  # the first pass makes the file system allocate the pages
        t = time.perf_counter()
        write_all()
        write_gbs = w.image_bytes / (time.perf_counter() - t) / 1e9
        cpu_t = torch.from_numpy(arr)
        ts = []
        for _ in range(5):
            e0, e1 = event_list(torch, 2)
            e0.record()
            cpu_t.copy_(bench.image[:buf_bytes], non_blocking=True)
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        d2h_gbs = buf_bytes / min(ts) / 1e6
        gms.gms_host_image_free(hptr)
        bd_capture = torch.zeros_like(bench.bd)
        gms.gms_capture_fd(bench.m, pipe, wfd, 0, bd_capture, bench.td)
        cstats = [gms.gms_capture_fd(bench.m, pipe, wfd, 0, bd_capture, bench.td) for _ in range(steps)]
        os.close(wfd)
        cbest = min(cstats, key=lambda s: s["total_seconds"])
        cgbs = w.payload_bytes / cbest["total_seconds"] / 1e9

        def file_ok():
            """What was written is what was there: a restore fed from the new file must digest to the recorded values."""
            rfd = os.open(path, os.O_RDONLY)
            try:
                bench.bd.zero_()
                gms.gms_restore_fd(bench.m, pipe, rfd, 0, bench.bd, bench.td)
            finally:
                os.close(rfd)
            gms.gms_verify(bench.m, bench.bd, bench.mm, bench.cap, bench.cnt)
            return bench.check() and bool(torch.equal(bench.bd, bd_capture))

        cok = file_ok()
        with open(path, "r+b") as f:  # so that the second pass cannot pass on what the first one wrote
            for a in range(0, w.image_bytes, 1 << 30):
                f.seek(a)
                f.write(bytes(min(1 << 20, w.image_bytes - a)))
        # the same with the writers storing through a shared mapping of the file (buffered writes to one file are
        # serialised by the kernel, stores into a mapping are not); yardstick: the same threads copying one pinned
        # buffer into a mapping of the file
        import mmap

        wfd = os.open(path, os.O_RDWR)
        hptr, _, arr = gms.gms_host_image_alloc(buf_bytes)

        def map_all():  # a fresh mapping every pass, as in the call: its pages have to be mapped in again
            mm = mmap.mmap(wfd, w.image_bytes)
            mapped = np.frombuffer(mm, dtype=np.uint8)

            def store(lo, o, n):
                mapped[lo + o:lo + o + n] = arr[o:o + n]

            with cf.ThreadPoolExecutor(n_readers) as ex:
                for lo in range(0, w.image_bytes, buf_bytes):
                    n = min(buf_bytes, w.image_bytes - lo)
                    for fu in [ex.submit(store, lo, o, min(slice_b, n - o)) for o in range(0, n, slice_b)]:
                        fu.result()
            del mapped
            mm.close()

        map_all()
        t = time.perf_counter()
        map_all()
        map_gbs = w.image_bytes / (time.perf_counter() - t) / 1e9
        gms.gms_host_image_free(hptr)
        gms.gms_pipe_mapped_writes(pipe, True)
        gms.gms_capture_fd(bench.m, pipe, wfd, 0, bd_capture, bench.td)
        mstats = [gms.gms_capture_fd(bench.m, pipe, wfd, 0, bd_capture, bench.td) for _ in range(steps)]
        gms.gms_pipe_mapped_writes(pipe, False)
        os.close(wfd)
        mbest = min(mstats, key=lambda s: s["total_seconds"])
        mgbs = w.payload_bytes / mbest["total_seconds"] / 1e9
        mbound = min(map_gbs, d2h_gbs)
        mok = file_ok() and mbest["mapped_io"] == 1
        cbound = min(write_gbs, d2h_gbs)
        line["capture_fd"] = {"value": cgbs, "unit": UNIT, "ms": cbest["total_seconds"] * 1e3, "bound": "storage_write" if write_gbs < d2h_gbs else "host_link",
                              "peak": cbound, "frac": cgbs / cbound, "writer_yardstick_gbs": write_gbs, "link_yardstick_gbs": d2h_gbs,
                              "peak_kind": "min(same writer threads and slicing emptying one pinned buffer into the same file with no producer; "
                                           "plain cudaMemcpyAsync D2H of one pinned buffer)", "pipe_stats_best": cbest, "parity_ok": bool(cok)}
        line["capture_fd_mapped"] = {"value": mgbs, "unit": UNIT, "ms": mbest["total_seconds"] * 1e3, "bound": "storage_write" if map_gbs < d2h_gbs else "host_link",
                                     "peak": mbound, "frac": mgbs / mbound, "writer_yardstick_gbs": map_gbs, "link_yardstick_gbs": d2h_gbs,
                                     "peak_kind": "min(same threads and slicing copying one pinned buffer into a shared mapping of the same file; "
                                                  "plain cudaMemcpyAsync D2H of one pinned buffer)", "pipe_stats_best": mbest,
                                     "parity_ok": bool(mok)}
        pipe.close()
        bench.close()
        return line
    finally:
        if os.path.exists(path):
            os.remove(path)


def unfused_comparison(torch, gms, bench, steps, warmup, index):
    """The same manifest step as four separate calls, on the same buffers (what the fused calls save)."""
    bench.set_fused(False)
    ue = measure(torch, gms, bench, steps, warmup, index)
    bench.set_fused(True)
    return {"step": ue["step"], "steps": steps, "ms_per_step": ue["ms_per_step"], "parity_ok": ue["parity_ok"],
            "phases_ms_median": {k: v["median_ms"] for k, v in ue["phases"].items()},
            "phases_ms_mean": {k: v["mean_ms"] for k, v in ue["phases"].items()}}


def release(torch):
    gc.collect()
    torch.cuda.synchronize()
    torch.cuda.empty_cache()


def compact(entry):
    """The few figures of a configuration that must survive truncation of the line."""
    r = entry["roofline"]
    c = {"ms": round(entry["ms_per_step"], 5), "gbs": round(entry["value"], 1), "frac": round(r["frac"], 4), "bound": r["bound"],
         "parity_ok": entry["parity_ok"], "sm_mhz": entry["clocks"].get("sm_mhz")}
    if "frac_of_datasheet_8TBps" in r:
        c["frac_8TBps"] = round(r["frac_of_datasheet_8TBps"], 4)
    if "mapped_frac" in r:
        c["mapped_frac"] = round(r["mapped_frac"], 4)
    if entry.get("cpu_baseline"):
        c["cpu_gbs"] = round(entry["cpu_baseline"]["value"], 3)
        c["cpu_cores"] = entry["cpu_baseline"]["cores"]
        if "all_cores" in entry["cpu_baseline"]:
            c["cpu_all_gbs"] = round(entry["cpu_baseline"]["all_cores"]["value"], 3)
            c["cpu_all_cores"] = entry["cpu_baseline"]["all_cores"]["cores"]
    c["phases_ms"] = {k: round(v.get("median_ms", v.get("mean_ms")), 5) for k, v in entry["phases"].items()}
    if entry.get("per_tensor_memcpy"):
        c["vs_per_tensor_memcpy"] = round(entry["per_tensor_memcpy"]["restore_speedup"], 2)
    if entry.get("manifest_build_ms") is not None:
        c["build_ms"] = round(entry["manifest_build_ms"], 3)
    return c


def main():
    args = parse_args()
    if args.impl == "reference":
        reference_arm(args)
        return
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
    want_cpu = rank == 0 and world == 1 and not args.no_cpu_baseline
    headline = args.workload or "8b"

    # ---- workloads that are not a device-resident manifest step
    if headline in ("host70b", "file"):
        if headline == "host70b":
            entry = run_host70b(args, torch, gms, W, dev, local_rank, want_cpu, args.cpu_seconds_other)
            line = {"metric": "host-sourced restore+digest GB/s", "value": entry["value"], "unit": UNIT, "n_gpus": 1,
                    "steps": entry["steps"], "warmup": 1, "ms_per_step": entry["ms_per_step"], "higher_is_better": True,
                    "scaling": "weak", "vs_baseline": None, "dtype": "u64", "data": "synthetic",
                    "config": {"workload": entry["workload"], "step": entry["step"], "l2": entry["l2"]},
                    "roofline": entry["roofline"], "clocks": entry["clocks"], "gpu_launches": entry["gpu_launches"],
                    "phases": entry["phases"], "one_shard_restore_s": entry["one_shard_restore_s"], "parity_ok": entry["parity_ok"],
                    "cpu_baseline": entry.get("cpu_baseline")}
        else:
            line = run_file(args, torch, gms, W, dev, local_rank, want_cpu)
        if rank == 0:
            print(json.dumps(line), flush=True)
        return

    # ---- the headline
    def build(name, fused=True):
        if name == "kv":
            return KvBench(torch, gms, W, dev, pool_bytes=args.kv_gb * 1e9)
        if name == "capture":
            return CaptureBench(torch, gms, W, dev, vmm=args.vmm)
        return ManifestBench(name, torch, gms, W, dev, fused=fused, vmm=args.vmm, shrink=args.shrink if name == "8b" else 1)

    bench = build(headline, fused=not args.unfused)
    if args.no_l2_flush and getattr(bench, "l2_flush", None) is not None:
        bench.l2_flush = None
    graphed = args.graph and type(bench) is ManifestBench
    entry = measure(torch, gms, bench, args.steps, args.warmup, local_rank, d, dev, graph=graphed)
    line = {
        "metric": METRIC, "value": entry["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": entry["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "u64", "data": "synthetic", "config": bench.config(), "roofline": entry["roofline"], "clocks": entry["clocks"],
        "gpu_launches": entry["gpu_launches"], "parity_ok": entry["parity_ok"],
        "phases_ms": {k: v["mean_ms"] for k, v in entry["phases"].items()},
        "phases_ms_median_best": {k: {"median": v.get("median_ms"), "best": v.get("best_ms")} for k, v in entry["phases"].items()},
        "geometry": gms.gms_launch_geometry(), "manifest_build_ms": entry.get("manifest_build_ms"),
    }
    if graphed:
        line["config"]["launch"] = f"CUDA graph replay ({bench.launches_per_step} kernel nodes per step)"
    ph = entry["phases"]
    if type(bench) is ManifestBench and not graphed:
        rk, dk = ("restore_verify", "digest_verify") if bench.fused else ("restore", "digest")
        line["restore_s"] = ph[rk]["mean_ms"] / 1e3
        line["restore_payload_gbs"] = bench.payload / ph[rk]["mean_ms"] / 1e6
        line["digest_read_gbs"] = bench.phase_bytes[dk] / ph[dk]["mean_ms"] / 1e6
        line["digest_frac_of_peak"] = line["digest_read_gbs"] / entry["roofline"]["peak"]
        line["digest_frac_of_8TBps"] = line["digest_read_gbs"] / DATASHEET_HBM_GBS
        y = per_tensor_memcpy_yardstick(torch, bench)
        if y:
            line["per_tensor_memcpy"] = {
                "ms": y[0], "host_issue_ms": y[1], "calls": y[2], "payload_gbs": bench.payload / y[0] / 1e6,
                "restore_speedup": y[0] / ph[rk]["mean_ms"],
                "note": "one cudaMemcpyAsync D2D per tensor on one stream, no digest (the launch-per-tensor yardstick)"}

    # ---- end to end: snapshot image in pinned host memory, verdict read back every step
    if not args.no_e2e and type(bench) is ManifestBench and bench.graph is None:
        try:
            line["e2e"] = e2e_leg(args, torch, gms, bench, d, dev)
        except gms.GmsError as ex:  # the host image could not be pinned on this machine
            line["e2e"] = None
            line["e2e_error"] = str(ex)[:300]
    elif not args.no_e2e:
        line["e2e"] = None
    if not args.no_e2e and type(bench) is CaptureBench:
        try:
            line["capture_to_host"] = capture_to_host_leg(torch, gms, bench)
        except gms.GmsError as ex:
            line["capture_to_host"] = {"error": str(ex)[:300]}

    if want_cpu and type(bench) in (ManifestBench, CaptureBench):
        fetch = lambda lo, hi: bench.image[lo:hi].cpu().numpy()
        line["cpu_baseline"] = cpu_baseline_manifest(bench.w, fetch, args.cpu_seconds, all_cores=True)
    elif want_cpu and type(bench) is KvBench:
        line["cpu_baseline"] = cpu_baseline_kv(bench.k, lambda n: bench.image[:n].cpu().numpy())
    if type(bench) is KvBench and not args.no_e2e:
        try:
            line["host_legs"] = kv_host_legs(torch, gms, bench)
        except gms.GmsError as ex:
            line["host_legs"] = {"error": str(ex)[:300]}

    # ---- all five configurations (single GPU, default invocation only)
    if args.workload is None and world == 1:
        entry["per_tensor_memcpy"] = line.get("per_tensor_memcpy")
        entry["unfused_step"] = unfused_comparison(torch, gms, bench, min(args.steps, 10), args.warmup, local_rank)
        line["unfused_step"] = entry["unfused_step"]
        entry["cpu_baseline"] = line.get("cpu_baseline")
        entry["e2e"] = line.get("e2e")
        configs = {"8b": entry}
        bench.close()
        del bench
        release(torch)
        def one_config(name):
            if name == "host70b":
                return run_host70b(args, torch, gms, W, dev, local_rank, want_cpu, args.cpu_seconds_other)
            b = build(name)
            steps = 50 if name == "tiny" else args.steps
            e = measure(torch, gms, b, steps, args.warmup, local_rank)
            if name != "kv":  # also the same work as four separate calls, and as one plain copy per tensor
                e["unfused_step"] = unfused_comparison(torch, gms, b, steps, args.warmup, local_rank)
                y = per_tensor_memcpy_yardstick(torch, b)
                if y:
                    r_ms = e["phases"]["restore_verify"]["mean_ms"]
                    e["per_tensor_memcpy"] = {"ms": y[0], "host_issue_ms": y[1], "calls": y[2], "restore_speedup": y[0] / r_ms,
                                              "note": "one cudaMemcpyAsync D2D per tensor on one stream, no digest, no verify"}
            if name == "tiny":
                e["note"] = ("latency-bound: 67 MB of traffic is 10 us at the HBM rate; what is measured is launch, "
                             "ramp-up and tail of a 148-CTA persistent kernel")
            if name == "kv" and not args.no_e2e:
                try:
                    e["host_legs"] = kv_host_legs(torch, gms, b)
                except gms.GmsError as ex:
                    e["host_legs"] = {"error": str(ex)[:300]}
            if want_cpu and name == "kv":
                e["cpu_baseline"] = cpu_baseline_kv(b.k, lambda n: b.image[:n].cpu().numpy())
            elif want_cpu:
                fetch = lambda lo, hi: b.image[lo:hi].cpu().numpy()
                e["cpu_baseline"] = cpu_baseline_manifest(b.w, fetch, args.cpu_seconds_other, all_cores=True)
            b.close()
            del b
            return e

        for name in CONFIG_ORDER:
            if name == "8b":
                continue
            try:  # a configuration that cannot run here (say, no room to pin 32 GiB) must not cost the others their line
                configs[name] = one_config(name)
            except Exception as ex:  # noqa: BLE001
                configs[name] = {"error": f"{type(ex).__name__}: {ex}"[:400], "parity_ok": False}
            release(torch)
        line["configs"] = {name: configs[name] for name in CONFIG_ORDER}
        line["config"]["all_five"] = {name: (compact(c) if "error" not in c else c) for name, c in line["configs"].items()}
        # ---- the inverse path and the service substrate on the 8B manifest: gms_capture into a device image and into a
        # pinned host image, and the headline step with the destinations in gms_service VMM slabs
        extra_steps = max(3, min(args.steps, 10))
        try:
            cb = CaptureBench(torch, gms, W, dev)
            ce = measure(torch, gms, cb, extra_steps, args.warmup, local_rank)
            line["capture"] = compact(ce)
            if not args.no_e2e:
                try:
                    line["capture"]["to_host"] = capture_to_host_leg(torch, gms, cb)
                except gms.GmsError as ex:
                    line["capture"]["to_host"] = {"error": str(ex)[:300]}
            cb.close()
            del cb
        except Exception as ex:  # noqa: BLE001
            line["capture"] = {"error": f"{type(ex).__name__}: {ex}"[:400], "parity_ok": False}
        release(torch)
        try:
            vb = ManifestBench("8b", torch, gms, W, dev, vmm=True)
            ve = measure(torch, gms, vb, extra_steps, args.warmup, local_rank)
            line["vmm_slabs"] = compact(ve)
            line["vmm_slabs"]["destinations"] = vb.config()["destinations"]
            vb.close()
            del vb
        except Exception as ex:  # noqa: BLE001
            line["vmm_slabs"] = {"error": f"{type(ex).__name__}: {ex}"[:400], "parity_ok": False}
        release(torch)
        # ---- the storage-fed legs (file -> pinned ring -> copy engine -> device, and back), a sixth entry beside the five
        if not args.no_file:
            try:
                import shutil

                need = W.llama3_8b_manifest().image_bytes + (1 << 30)
                if shutil.disk_usage(args.file_dir).free < need:
                    raise RuntimeError(f"{args.file_dir} has less than {need} bytes free")
                f = run_file(args, torch, gms, W, dev, local_rank, want_cpu=False, steps_cap=2)
                keep = ("value", "unit", "steps", "ms_per_step", "roofline", "pipe_stats_best", "parity_ok", "capture_fd", "capture_fd_mapped")
                line["storage_fed"] = {k: f[k] for k in keep if k in f}
                line["storage_fed"]["workload"] = f["config"]["workload"]
                line["storage_fed"]["file_system"] = f["config"]["file_system"]
            except Exception as ex:  # noqa: BLE001  (no room for the file, say: the line stands without this entry)
                line["storage_fed"] = {"error": f"{type(ex).__name__}: {ex}"[:400], "parity_ok": False}
            release(torch)
        # last key of the line, so that it survives a reader that keeps only the end of the output
        line["five_configs"] = "; ".join(
            (f"{n}: {c['ms']} ms {c['gbs']} GB/s frac {c['frac']} ({c['bound']}) parity {'ok' if c['parity_ok'] else 'FAILED'}"
             + (f" cpu {c['cpu_gbs']} GB/s x{c['cpu_cores']}" if "cpu_gbs" in c else "")
             + (f", {c['cpu_all_gbs']} x{c['cpu_all_cores']}" if "cpu_all_gbs" in c else "")) if "error" not in c else f"{n}: {c['error'][:80]}"
            for n, c in line["config"]["all_five"].items())
        sf = line.get("storage_fed")
        if sf and "error" not in sf:
            line["five_configs"] += (f"; file-fed restore ({sf['file_system']}): {round(sf['value'], 1)} GB/s frac {round(sf['roofline']['frac'], 3)} "
                                     f"({sf['roofline']['bound']}) parity {'ok' if sf['parity_ok'] else 'FAILED'}")
    else:
        bench.close()

    if rank == 0:
        print(json.dumps(line), flush=True)
    if use_dist:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
