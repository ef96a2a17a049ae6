"""Thin ctypes binding of the C ABI in ``include/gms.h`` -- argument marshalling only.

Every function has the name and meaning of the C entry point.  Device buffers
may be passed as ``torch`` tensors (their ``data_ptr()`` is taken), as ints, or
as ``None`` where the C ABI accepts NULL.  Nothing here computes anything: if
the shared library is missing or a call fails, an exception is raised -- there
is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libgms.so")

BLOCK_BYTES = 4096
OK = 0
ERR_NULL, ERR_ALIGN, ERR_RANGE, ERR_OVERLAP, ERR_DUP_ID, ERR_NOMEM = -1, -2, -3, -4, -5, -6
ERR_CUDA, ERR_KIND, ERR_TIMEOUT, ERR_STATE, ERR_ARG, ERR_TOO_LARGE, ERR_IO = -7, -8, -9, -10, -11, -12, -13
NOALLOC_MAX_BLOCKS = 4194304
SRC_DEVICE, SRC_HOST_MAPPED = 0, 1
BUILD_HOST_ONLY = 1
BUILD_SELFTEST_STALL = 2  # test suites only: one warp's first wait runs out (see include/gms.h)
DEV_TIMEOUT = 1  # bit of the device status word

# numpy view of gms_entry / gms_mismatch (32 and 16 bytes)
ENTRY_DTYPE = np.dtype([("tensor_id", "<u8"), ("src_offset", "<u8"), ("dst", "<u8"), ("nbytes", "<u8")])
MISMATCH_DTYPE = np.dtype([("tensor_id", "<u8"), ("block", "<u8")])
KV_MISMATCH_DTYPE = np.dtype([("block_id", "<u4"), ("plane", "<u4"), ("sub_block", "<u4"), ("list_pos", "<u4")])

EXPORTS = (
    "gms_manifest_build", "gms_manifest_destroy", "gms_manifest_info", "gms_manifest_block_base",
    "gms_manifest_chunk_count", "gms_manifest_chunk", "gms_manifest_set_expected", "gms_restore", "gms_capture", "gms_digest",
    "gms_verify", "gms_digest_verify", "gms_restore_verify", "gms_verify_tensors", "gms_verify_flat_noalloc", "gms_last_device_status", "gms_kv_restore", "gms_kv_capture", "gms_kv_digest", "gms_kv_verify", "gms_host_image_alloc", "gms_host_image_free",
    "gms_pipe_create", "gms_pipe_direct_io", "gms_pipe_mapped_writes", "gms_pipe_destroy", "gms_restore_fd", "gms_capture_fd", "gms_stage_create", "gms_stage_destroy", "gms_restore_staged",
    "gms_service_create", "gms_service_destroy", "gms_service_acquire_rw", "gms_service_alloc", "gms_service_commit",
    "gms_service_abort", "gms_service_acquire_ro", "gms_service_release_ro", "gms_service_info", "gms_service_access",
    "gms_service_detach", "gms_service_reattach", "gms_service_release_pages", "gms_service_back_pages",
    "gms_service_slab", "gms_service_export_fd", "gms_import_create", "gms_import_address", "gms_import_destroy",
    "gms_launch_geometry", "gms_kernel_launches", "gms_set_device", "gms_strerror", "gms_last_cuda_error", "gms_version",
)


class GmsError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        text = lib().gms_strerror(status).decode()
        if status == ERR_CUDA:
            text += " -- " + lib().gms_last_cuda_error().decode()
        super().__init__(f"{where}: {text} ({status})")


class KvPool(C.Structure):
    _fields_ = [("base", C.c_void_p), ("plane_stride", C.c_uint64), ("block_stride", C.c_uint64),
                ("n_planes", C.c_uint32), ("n_blocks", C.c_uint32), ("block_bytes", C.c_uint32), ("flags", C.c_uint32)]


KV_IMAGE_BY_ID = 1


_lib = None


def lib():
    """Loads ``libgms.so`` (built by ``paper_2609_25451_b200.build``); raises if it is absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2609_25451_b200.build` (needs nvcc)")
        L = C.CDLL(LIB_PATH)
        p, u64, u32, i = C.c_void_p, C.c_uint64, C.c_uint32, C.c_int
        pp = C.POINTER(C.c_void_p)
        pu64, pu32 = C.POINTER(C.c_uint64), C.POINTER(C.c_uint32)
        sig = {
            "gms_manifest_build": (i, [p, C.c_size_t, u64, u32, pp]),
            "gms_manifest_destroy": (i, [p]),
            "gms_manifest_info": (i, [p, pu64, pu64, pu64]),
            "gms_manifest_block_base": (i, [p, C.c_size_t, pu64]),
            "gms_manifest_chunk_count": (i, [p, pu64]),
            "gms_manifest_chunk": (i, [p, u64, pu64, pu64, pu64]),
            "gms_manifest_set_expected": (i, [p, p, p]),
            "gms_restore": (i, [p, p, u32, p, p, p]),
            "gms_capture": (i, [p, p, u32, p, p, p]),
            "gms_digest": (i, [p, p, p, p]),
            "gms_verify": (i, [p, p, p, u32, p, p]),
            "gms_digest_verify": (i, [p, p, p, p, u32, p, p]),
            "gms_restore_verify": (i, [p, p, u32, p, p, p, u32, p, p]),
            "gms_verify_tensors": (i, [p, p, p, p]),
            "gms_verify_flat_noalloc": (i, [p, p, u64, u64, p, u32, p, p]),
            "gms_last_device_status": (i, [p, p, pu64]),
            "gms_kv_restore": (i, [C.POINTER(KvPool), p, u64, u64, u32, p, u32, p, p, p, p]),
            "gms_kv_capture": (i, [C.POINTER(KvPool), p, u64, u64, u32, p, u32, p, p, p, p]),
            "gms_kv_digest": (i, [C.POINTER(KvPool), p, u32, p, p, p, p]),
            "gms_kv_verify": (i, [C.POINTER(KvPool), p, u32, p, p, p, u32, p, p, p]),
            "gms_host_image_alloc": (i, [u64, pp, pp]),
            "gms_host_image_free": (i, [p]),
            "gms_pipe_create": (i, [u32, u64, u32, pp]),
            "gms_pipe_direct_io": (i, [p, i]),
            "gms_pipe_mapped_writes": (i, [p, i]),
            "gms_pipe_destroy": (i, [p]),
            "gms_restore_fd": (i, [p, p, i, u64, p, p, p, p]),
            "gms_capture_fd": (i, [p, p, i, u64, p, p, p, p]),
            "gms_stage_create": (i, [u32, u64, pp]),
            "gms_stage_destroy": (i, [p]),
            "gms_restore_staged": (i, [p, p, p, p, p, p]),
            "gms_service_create": (i, [u64, u32, pp]),
            "gms_service_destroy": (i, [p]),
            "gms_service_acquire_rw": (i, [p]),
            "gms_service_alloc": (i, [p, u64, pp]),
            "gms_service_commit": (i, [p]),
            "gms_service_abort": (i, [p]),
            "gms_service_acquire_ro": (i, [p]),
            "gms_service_release_ro": (i, [p]),
            "gms_service_info": (i, [p, p]),
            "gms_service_access": (i, [p, p, pu32]),
            "gms_service_detach": (i, [p]),
            "gms_service_reattach": (i, [p]),
            "gms_service_release_pages": (i, [p]),
            "gms_service_back_pages": (i, [p]),
            "gms_service_slab": (i, [p, u64, p]),
            "gms_service_export_fd": (i, [p, u64, p]),
            "gms_import_create": (i, [p, p, C.c_size_t, u32, p]),
            "gms_import_address": (i, [p, C.c_size_t, p]),
            "gms_import_destroy": (i, [p]),
            "gms_launch_geometry": (i, [pu32, pu32, pu32]),
            "gms_kernel_launches": (u64, []),
            "gms_set_device": (i, [i]),
            "gms_strerror": (C.c_char_p, [i]),
            "gms_last_cuda_error": (C.c_char_p, []),
            "gms_version": (u32, []),
        }
        for name, (res, args) in sig.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


def _dev(x):
    """Address of a device buffer: torch tensor, int or None."""
    if x is None:
        return None
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    return int(x)


def _stream(stream):
    if stream is None:
        import torch

        return torch.cuda.current_stream().cuda_stream if torch.cuda.is_available() else None
    return getattr(stream, "cuda_stream", stream)


def _check(rc: int, where: str):
    if rc != OK:
        raise GmsError(rc, where)


def make_entries(rows) -> np.ndarray:
    """rows: iterable of (tensor_id, src_offset, dst_address, nbytes) -> gms_entry array."""
    rows = list(rows)
    a = np.zeros(len(rows), dtype=ENTRY_DTYPE)
    for k, r in enumerate(rows):
        a[k] = tuple(int(v) for v in r)
    return a


class Manifest:
    """Owner of a ``gms_manifest*``; destroyed on ``close()`` / garbage collection."""

    def __init__(self, handle):
        self.handle = handle
        n, nb, pay = C.c_uint64(), C.c_uint64(), C.c_uint64()
        _check(lib().gms_manifest_info(handle, C.byref(n), C.byref(nb), C.byref(pay)), "gms_manifest_info")
        self.n_tensors, self.n_blocks, self.payload_bytes = n.value, nb.value, pay.value

    def close(self):
        if self.handle:
            lib().gms_manifest_destroy(self.handle)
            self.handle = None

    __del__ = close


def gms_manifest_build(entries, image_bytes: int, flags: int = 0) -> Manifest:
    e = np.ascontiguousarray(entries, dtype=ENTRY_DTYPE)
    out = C.c_void_p()
    rc = lib().gms_manifest_build(e.ctypes.data if len(e) else None, len(e), int(image_bytes), int(flags), C.byref(out))
    _check(rc, "gms_manifest_build")
    return Manifest(out.value)


def gms_manifest_block_base(m: Manifest, entry_index: int) -> int:
    v = C.c_uint64()
    _check(lib().gms_manifest_block_base(m.handle, entry_index, C.byref(v)), "gms_manifest_block_base")
    return v.value


def gms_manifest_chunk_count(m: Manifest) -> int:
    v = C.c_uint64()
    _check(lib().gms_manifest_chunk_count(m.handle, C.byref(v)), "gms_manifest_chunk_count")
    return v.value


def gms_manifest_chunk(m: Manifest, i: int):
    """Returns (entry_index, tensor_byte_offset, nbytes) of work-list chunk ``i``."""
    a, b, c = C.c_uint64(), C.c_uint64(), C.c_uint64()
    _check(lib().gms_manifest_chunk(m.handle, i, C.byref(a), C.byref(b), C.byref(c)), "gms_manifest_chunk")
    return a.value, b.value, c.value


def gms_manifest_set_expected(m: Manifest, d_block_digests, stream=None):
    _check(lib().gms_manifest_set_expected(m.handle, _dev(d_block_digests), _stream(stream)), "gms_manifest_set_expected")


def gms_restore(m: Manifest, image, image_kind: int, d_block_digests, d_tensor_digests, stream=None):
    _check(lib().gms_restore(m.handle, _dev(image), image_kind, _dev(d_block_digests), _dev(d_tensor_digests),
                             _stream(stream)), "gms_restore")


def gms_capture(m: Manifest, image, image_kind: int, d_block_digests, d_tensor_digests, stream=None):
    _check(lib().gms_capture(m.handle, _dev(image), image_kind, _dev(d_block_digests), _dev(d_tensor_digests),
                             _stream(stream)), "gms_capture")


def gms_digest(m: Manifest, d_block_digests, d_tensor_digests, stream=None):
    _check(lib().gms_digest(m.handle, _dev(d_block_digests), _dev(d_tensor_digests), _stream(stream)), "gms_digest")


def gms_verify(m: Manifest, d_block_digests, d_out, cap: int, d_count, stream=None):
    _check(lib().gms_verify(m.handle, _dev(d_block_digests), _dev(d_out), cap, _dev(d_count), _stream(stream)), "gms_verify")


def gms_digest_verify(m: Manifest, d_block_digests, d_tensor_digests, d_out, cap: int, d_count, stream=None):
    _check(lib().gms_digest_verify(m.handle, _dev(d_block_digests), _dev(d_tensor_digests), _dev(d_out), cap, _dev(d_count),
                                   _stream(stream)), "gms_digest_verify")


def gms_restore_verify(m: Manifest, image, image_kind: int, d_block_digests, d_tensor_digests, d_out, cap: int, d_count,
                       stream=None):
    _check(lib().gms_restore_verify(m.handle, _dev(image), image_kind, _dev(d_block_digests), _dev(d_tensor_digests),
                                    _dev(d_out), cap, _dev(d_count), _stream(stream)), "gms_restore_verify")


def gms_verify_tensors(m: Manifest, d_block_digests, d_tensor_counts, stream=None):
    _check(lib().gms_verify_tensors(m.handle, _dev(d_block_digests), _dev(d_tensor_counts), _stream(stream)),
           "gms_verify_tensors")


def gms_verify_flat_noalloc(d_computed, d_expected, n_blocks: int, tensor_id: int, d_out, cap: int, d_count, stream=None):
    """Allocation-free comparison of two device digest arrays; see include/gms.h for who needs it."""
    _check(lib().gms_verify_flat_noalloc(_dev(d_computed), _dev(d_expected), int(n_blocks), int(tensor_id), _dev(d_out),
                                         cap, _dev(d_count), _stream(stream)), "gms_verify_flat_noalloc")


def gms_last_device_status(m: Manifest, stream=None) -> int:
    w = C.c_uint64()
    _check(lib().gms_last_device_status(m.handle, _stream(stream), C.byref(w)), "gms_last_device_status")
    return w.value


def gms_kv_restore(pool: KvPool, image, img_plane_stride: int, img_slot_stride: int, image_kind: int, d_block_ids,
                   n_sel: int, d_block_digests, d_kv_digests, d_status, stream=None):
    _check(lib().gms_kv_restore(C.byref(pool), _dev(image), img_plane_stride, img_slot_stride, image_kind,
                                _dev(d_block_ids), n_sel, _dev(d_block_digests), _dev(d_kv_digests), _dev(d_status),
                                _stream(stream)), "gms_kv_restore")


def gms_kv_capture(pool: KvPool, image, img_plane_stride: int, img_slot_stride: int, image_kind: int, d_block_ids,
                   n_sel: int, d_block_digests, d_kv_digests, d_status, stream=None):
    _check(lib().gms_kv_capture(C.byref(pool), _dev(image), img_plane_stride, img_slot_stride, image_kind,
                                _dev(d_block_ids), n_sel, _dev(d_block_digests), _dev(d_kv_digests), _dev(d_status),
                                _stream(stream)), "gms_kv_capture")


def gms_kv_digest(pool: KvPool, d_block_ids, n_sel: int, d_block_digests, d_kv_digests, d_status, stream=None):
    _check(lib().gms_kv_digest(C.byref(pool), _dev(d_block_ids), n_sel, _dev(d_block_digests), _dev(d_kv_digests),
                               _dev(d_status), _stream(stream)), "gms_kv_digest")


def kv_verify_scratch_words(n_slots: int) -> int:
    """GMS_KV_VERIFY_SCRATCH_WORDS of include/gms.h: u32 words of caller-owned working memory for gms_kv_verify."""
    return (int(n_slots) + 2047) // 2048 + 1


def gms_kv_verify(pool: KvPool, d_block_ids, n_sel: int, d_computed, d_expected, d_out, cap: int, d_count, d_scratch,
                  stream=None):
    _check(lib().gms_kv_verify(C.byref(pool), _dev(d_block_ids), n_sel, _dev(d_computed), _dev(d_expected), _dev(d_out), cap,
                               _dev(d_count), _dev(d_scratch), _stream(stream)), "gms_kv_verify")


def gms_host_image_alloc(nbytes: int):
    """Returns (host_ptr, device_view, numpy uint8 array over the pinned mapping)."""
    h, d = C.c_void_p(), C.c_void_p()
    _check(lib().gms_host_image_alloc(int(nbytes), C.byref(h), C.byref(d)), "gms_host_image_alloc")
    arr = np.ctypeslib.as_array((C.c_uint8 * int(nbytes)).from_address(h.value))
    return h.value, d.value, arr


def gms_host_image_free(host_ptr: int):
    _check(lib().gms_host_image_free(host_ptr), "gms_host_image_free")


class PipeStats(C.Structure):
    _fields_ = [("windows", C.c_uint64), ("bytes_read", C.c_uint64), ("wait_read_seconds", C.c_double),
                ("wait_gpu_seconds", C.c_double), ("total_seconds", C.c_double), ("direct_io", C.c_uint32),
                ("copy_engine", C.c_uint32), ("mapped_io", C.c_uint32), ("reserved", C.c_uint32)]


class Pipe:
    """Owner of a ``gms_pipe*`` (ring of pinned buffers + reader threads)."""

    def __init__(self, handle):
        self.handle = handle

    def close(self):
        if self.handle:
            lib().gms_pipe_destroy(self.handle)
            self.handle = None

    __del__ = close


def gms_pipe_create(n_buffers: int, buffer_bytes: int, n_readers: int) -> Pipe:
    out = C.c_void_p()
    _check(lib().gms_pipe_create(n_buffers, int(buffer_bytes), n_readers, C.byref(out)), "gms_pipe_create")
    return Pipe(out.value)


def gms_pipe_direct_io(pipe: Pipe, enable: bool):
    _check(lib().gms_pipe_direct_io(pipe.handle, 1 if enable else 0), "gms_pipe_direct_io")


def gms_pipe_mapped_writes(pipe: Pipe, enable: bool):
    _check(lib().gms_pipe_mapped_writes(pipe.handle, 1 if enable else 0), "gms_pipe_mapped_writes")


def gms_restore_fd(m: Manifest, pipe: Pipe, fd: int, file_offset: int, d_block_digests, d_tensor_digests, stream=None) -> dict:
    """Synchronous; returns the call's statistics as a dict."""
    st = PipeStats()
    _check(lib().gms_restore_fd(m.handle, pipe.handle, int(fd), int(file_offset), _dev(d_block_digests),
                                _dev(d_tensor_digests), _stream(stream), C.byref(st)), "gms_restore_fd")
    return {k: getattr(st, k) for k, _ in PipeStats._fields_}


def gms_capture_fd(m: Manifest, pipe: Pipe, fd: int, file_offset: int, d_block_digests, d_tensor_digests, stream=None) -> dict:
    """Synchronous; returns the call's statistics as a dict (``bytes_read`` counts the bytes written)."""
    st = PipeStats()
    _check(lib().gms_capture_fd(m.handle, pipe.handle, int(fd), int(file_offset), _dev(d_block_digests),
                                _dev(d_tensor_digests), _stream(stream), C.byref(st)), "gms_capture_fd")
    return {k: getattr(st, k) for k, _ in PipeStats._fields_}


class Stage:
    """Owner of a ``gms_stage*`` (device staging ring fed by the copy engine)."""

    def __init__(self, handle):
        self.handle = handle

    def close(self):
        if self.handle:
            lib().gms_stage_destroy(self.handle)
            self.handle = None

    __del__ = close


def gms_stage_create(n_buffers: int, buffer_bytes: int) -> Stage:
    out = C.c_void_p()
    _check(lib().gms_stage_create(n_buffers, int(buffer_bytes), C.byref(out)), "gms_stage_create")
    return Stage(out.value)


def gms_restore_staged(m: Manifest, stage: Stage, host_image, d_block_digests, d_tensor_digests, stream=None):
    _check(lib().gms_restore_staged(m.handle, stage.handle, _dev(host_image), _dev(d_block_digests), _dev(d_tensor_digests),
                                    _stream(stream)), "gms_restore_staged")


STATE_EMPTY, STATE_RW, STATE_COMMITTED, STATE_RO = 0, 1, 2, 3
SERVICE_DRY_RUN = 1


class ServiceStats(C.Structure):
    _fields_ = [("state", C.c_uint32), ("readers", C.c_uint32), ("n_slabs", C.c_uint64), ("n_dedicated", C.c_uint64),
                ("slab_bytes", C.c_uint64), ("bytes_reserved", C.c_uint64), ("bytes_allocated", C.c_uint64),
                ("attached", C.c_uint32), ("backed", C.c_uint32)]


class Service:
    """Owner of a ``gms_service*``."""

    def __init__(self, handle):
        self.handle = handle

    def close(self):
        if self.handle:
            lib().gms_service_destroy(self.handle)
            self.handle = None

    __del__ = close


def gms_service_create(slab_bytes: int = 0, flags: int = 0) -> Service:
    out = C.c_void_p()
    _check(lib().gms_service_create(int(slab_bytes), flags, C.byref(out)), "gms_service_create")
    return Service(out.value)


def gms_service_acquire_rw(s: Service):
    _check(lib().gms_service_acquire_rw(s.handle), "gms_service_acquire_rw")


def gms_service_alloc(s: Service, nbytes: int) -> int:
    p = C.c_void_p()
    _check(lib().gms_service_alloc(s.handle, int(nbytes), C.byref(p)), "gms_service_alloc")
    return p.value


def gms_service_commit(s: Service):
    _check(lib().gms_service_commit(s.handle), "gms_service_commit")


def gms_service_abort(s: Service):
    _check(lib().gms_service_abort(s.handle), "gms_service_abort")


def gms_service_acquire_ro(s: Service):
    _check(lib().gms_service_acquire_ro(s.handle), "gms_service_acquire_ro")


def gms_service_release_ro(s: Service):
    _check(lib().gms_service_release_ro(s.handle), "gms_service_release_ro")


def gms_service_info(s: Service) -> dict:
    st = ServiceStats()
    _check(lib().gms_service_info(s.handle, C.byref(st)), "gms_service_info")
    return {k: getattr(st, k) for k, _ in ServiceStats._fields_}


def gms_service_access(s: Service, dptr: int) -> bool:
    """True if the address is currently mapped writable."""
    w = C.c_uint32()
    _check(lib().gms_service_access(s.handle, int(dptr), C.byref(w)), "gms_service_access")
    return bool(w.value)


def gms_service_detach(s: Service):
    _check(lib().gms_service_detach(s.handle), "gms_service_detach")


def gms_service_reattach(s: Service):
    _check(lib().gms_service_reattach(s.handle), "gms_service_reattach")


def gms_service_release_pages(s: Service):
    _check(lib().gms_service_release_pages(s.handle), "gms_service_release_pages")


def gms_service_back_pages(s: Service):
    _check(lib().gms_service_back_pages(s.handle), "gms_service_back_pages")


def gms_launch_geometry():
    g, w, s = C.c_uint32(), C.c_uint32(), C.c_uint32()
    _check(lib().gms_launch_geometry(C.byref(g), C.byref(w), C.byref(s)), "gms_launch_geometry")
    return {"grid_ctas": g.value, "warps_per_cta": w.value, "smem_bytes": s.value}


def gms_kernel_launches() -> int:
    return int(lib().gms_kernel_launches())


def gms_set_device(device: int):
    _check(lib().gms_set_device(int(device)), "gms_set_device")


def gms_strerror(status: int) -> str:
    return lib().gms_strerror(status).decode()


def gms_version() -> int:
    return lib().gms_version()


# ---------------------------------------------------------------- across processes
SERVICE_SHAREABLE = 2
IMPORT_WRITABLE, IMPORT_SAME_ADDRESS = 1, 2


class SlabInfo(C.Structure):
    _fields_ = [("address", C.c_uint64), ("bytes", C.c_uint64), ("dedicated", C.c_uint32), ("reserved", C.c_uint32)]


def gms_service_slab(s: Service, index: int) -> dict:
    info = SlabInfo()
    _check(lib().gms_service_slab(s.handle, int(index), C.byref(info)), "gms_service_slab")
    return {"address": info.address, "bytes": info.bytes, "dedicated": info.dedicated}


def gms_service_export_fd(s: Service, index: int) -> int:
    """A new file descriptor for the slab (send it with SCM_RIGHTS, then close it)."""
    fd = C.c_int(-1)
    _check(lib().gms_service_export_fd(s.handle, int(index), C.byref(fd)), "gms_service_export_fd")
    return fd.value


class Import:
    """Owner of a ``gms_import*`` (slabs of another process's service mapped into this one)."""

    def __init__(self, handle, n):
        self.handle, self.n = handle, n

    def address(self, index: int) -> int:
        p = C.c_void_p()
        _check(lib().gms_import_address(self.handle, int(index), C.byref(p)), "gms_import_address")
        return p.value

    def close(self):
        if self.handle:
            lib().gms_import_destroy(self.handle)
            self.handle = None

    __del__ = close


def gms_import_create(fds, slabs, flags: int = 0) -> Import:
    """``slabs``: the dicts of gms_service_slab, in the order of ``fds``."""
    n = len(fds)
    cf = (C.c_int * max(n, 1))(*[int(f) for f in fds])
    cs = (SlabInfo * max(n, 1))()
    for k, sl in enumerate(slabs):
        cs[k].address, cs[k].bytes, cs[k].dedicated = int(sl["address"]), int(sl["bytes"]), int(sl.get("dedicated", 0))
    out = C.c_void_p()
    _check(lib().gms_import_create(cf, cs, n, flags, C.byref(out)), "gms_import_create")
    return Import(out.value, n)
