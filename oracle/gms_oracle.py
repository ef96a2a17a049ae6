"""ctypes face of the CPU oracle (``gms_oracle.c``).

TEST INFRASTRUCTURE ONLY: the test-suite, the smoke check and the benchmark's
CPU-baseline leg may import this; the product package never does, and this
module imports nothing from the product package.

Arrays are numpy arrays on the host.  A "record" is a numpy structured array
with fields ``tensor_id, src_offset, dst_offset, nbytes`` (all uint64): the
host-side analogue of the library's layout record, with the destination given
as an offset into one host slab instead of a device pointer.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gms_oracle.c")
_LIB = os.path.join(_HERE, "libgms_oracle.so")

ENTRY_DTYPE = np.dtype(
    [("tensor_id", "<u8"), ("src_offset", "<u8"), ("dst_offset", "<u8"), ("nbytes", "<u8")], align=False
)
MISMATCH_DTYPE = np.dtype([("tensor_id", "<u8"), ("block", "<u8")], align=False)
KV_MISMATCH_DTYPE = np.dtype([("block_id", "<u4"), ("plane", "<u4"), ("sub_block", "<u4"), ("list_pos", "<u4")], align=False)

OK, ERR_NULL, ERR_ALIGN, ERR_RANGE, ERR_OVERLAP, ERR_DUP_ID = 0, -1, -2, -3, -4, -5
BLOCK = 4096


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C, -O2); returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-std=c11", "-O2", "-fPIC", "-shared", "-Wall", "-Wextra", "-o", _LIB, _SRC]
        )
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        u64, p = C.c_uint64, C.c_void_p
        L.gmso_mix.restype = u64
        L.gmso_mix.argtypes = [u64]
        L.gmso_block_digest.restype = u64
        L.gmso_block_digest.argtypes = [p, C.c_size_t]
        L.gmso_num_blocks.restype = u64
        L.gmso_num_blocks.argtypes = [u64]
        L.gmso_tensor_digest.restype = u64
        L.gmso_tensor_digest.argtypes = [p, u64, p]
        L.gmso_validate.restype = C.c_int
        L.gmso_validate.argtypes = [p, C.c_size_t, u64, u64]
        L.gmso_block_bases.restype = u64
        L.gmso_block_bases.argtypes = [p, C.c_size_t, p]
        L.gmso_restore.restype = C.c_int
        L.gmso_restore.argtypes = [p, C.c_size_t, p, u64, p, u64, p, p]
        L.gmso_capture.restype = C.c_int
        L.gmso_capture.argtypes = [p, C.c_size_t, p, u64, p, u64, p, p]
        L.gmso_kv_capture.restype = C.c_int
        L.gmso_kv_capture.argtypes = [p, u64, u64, C.c_uint32, C.c_uint32, C.c_uint32, p, u64, u64, p, C.c_uint32, p, p, p]
        L.gmso_digest.restype = C.c_int
        L.gmso_digest.argtypes = [p, C.c_size_t, p, u64, p, p]
        L.gmso_verify.restype = u64
        L.gmso_verify.argtypes = [p, C.c_size_t, p, p, p, u64]
        L.gmso_kv_digest.restype = C.c_int
        L.gmso_kv_digest.argtypes = [p, u64, u64, C.c_uint32, C.c_uint32, C.c_uint32, p, C.c_uint32, p, p, p]
        L.gmso_kv_verify.restype = u64
        L.gmso_kv_verify.argtypes = [C.c_uint32, C.c_uint32, C.c_uint32, p, C.c_uint32, p, p, p, u64]
        L.gmso_kv_restore.restype = C.c_int
        L.gmso_kv_restore.argtypes = [p, u64, u64, C.c_uint32, C.c_uint32, C.c_uint32, p, u64, u64, p, C.c_uint32, p, p, p]
        _lib = L
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data


def _bytes_view(a) -> np.ndarray:
    a = np.ascontiguousarray(a)
    return a.view(np.uint8).reshape(-1)


def make_record(rows) -> np.ndarray:
    """rows: iterable of (tensor_id, src_offset, dst_offset, nbytes)."""
    rows = list(rows)
    rec = np.zeros(len(rows), dtype=ENTRY_DTYPE)
    for i, r in enumerate(rows):
        rec[i] = tuple(int(v) for v in r)
    return rec


def mix(z: int) -> int:
    return int(lib().gmso_mix(C.c_uint64(z & (2**64 - 1))))


def block_digest(data) -> int:
    b = _bytes_view(np.frombuffer(bytes(data), dtype=np.uint8) if isinstance(data, (bytes, bytearray)) else data)
    assert b.size <= BLOCK
    return int(lib().gmso_block_digest(_ptr(b) if b.size else None, b.size))


def num_blocks(nbytes: int) -> int:
    return int(lib().gmso_num_blocks(int(nbytes)))


def tensor_digest(data):
    """Returns (T, block_digests ndarray)."""
    b = _bytes_view(np.frombuffer(bytes(data), dtype=np.uint8) if isinstance(data, (bytes, bytearray)) else data)
    nb = num_blocks(b.size)
    bd = np.zeros(nb, dtype=np.uint64)
    T = lib().gmso_tensor_digest(_ptr(b) if b.size else None, b.size, _ptr(bd) if nb else None)
    return int(T), bd


def validate(record: np.ndarray, image_bytes: int, dst_bytes: int) -> int:
    record = np.ascontiguousarray(record, dtype=ENTRY_DTYPE)
    return int(lib().gmso_validate(_ptr(record), len(record), int(image_bytes), int(dst_bytes)))


def block_bases(record: np.ndarray):
    """Returns (first block of each tensor, total blocks)."""
    record = np.ascontiguousarray(record, dtype=ENTRY_DTYPE)
    base = np.zeros(len(record), dtype=np.uint64)
    total = lib().gmso_block_bases(_ptr(record), len(record), _ptr(base))
    return base, int(total)


def restore(record: np.ndarray, image: np.ndarray, dst: np.ndarray):
    """Scatter ``image`` into the host slab ``dst`` (modified in place).

    Returns (status, block_digests, tensor_digests).
    """
    record = np.ascontiguousarray(record, dtype=ENTRY_DTYPE)
    img, d = _bytes_view(image), dst.view(np.uint8).reshape(-1)
    assert d.flags.c_contiguous and d.flags.writeable
    _, nb = block_bases(record)
    bd, td = np.zeros(nb, dtype=np.uint64), np.zeros(len(record), dtype=np.uint64)
    rc = lib().gmso_restore(_ptr(record), len(record), _ptr(img), img.size, _ptr(d), d.size, _ptr(bd), _ptr(td))
    return int(rc), bd, td


def capture(record: np.ndarray, image: np.ndarray, dst: np.ndarray):
    """Gather the host slab ``dst`` into ``image`` (modified in place).

    Returns (status, block_digests, tensor_digests).
    """
    record = np.ascontiguousarray(record, dtype=ENTRY_DTYPE)
    img, d = image.view(np.uint8).reshape(-1), _bytes_view(dst)
    assert img.flags.c_contiguous and img.flags.writeable
    _, nb = block_bases(record)
    bd, td = np.zeros(nb, dtype=np.uint64), np.zeros(len(record), dtype=np.uint64)
    rc = lib().gmso_capture(_ptr(record), len(record), _ptr(img), img.size, _ptr(d), d.size, _ptr(bd), _ptr(td))
    return int(rc), bd, td


def digest(record: np.ndarray, dst: np.ndarray):
    """Digest the destinations in place.  Returns (status, block_digests, tensor_digests)."""
    record = np.ascontiguousarray(record, dtype=ENTRY_DTYPE)
    d = _bytes_view(dst)
    _, nb = block_bases(record)
    bd, td = np.zeros(nb, dtype=np.uint64), np.zeros(len(record), dtype=np.uint64)
    rc = lib().gmso_digest(_ptr(record), len(record), _ptr(d), d.size, _ptr(bd), _ptr(td))
    return int(rc), bd, td


def verify(record: np.ndarray, computed: np.ndarray, expected: np.ndarray, cap: int):
    """Returns (count, mismatches[:min(count, cap)])."""
    record = np.ascontiguousarray(record, dtype=ENTRY_DTYPE)
    computed = np.ascontiguousarray(computed, dtype=np.uint64)
    expected = np.ascontiguousarray(expected, dtype=np.uint64)
    assert computed.size == expected.size
    out = np.zeros(max(cap, 1), dtype=MISMATCH_DTYPE)
    n = int(lib().gmso_verify(_ptr(record), len(record), _ptr(computed), _ptr(expected), _ptr(out), int(cap)))
    return n, out[: min(n, cap)].copy()


def kv_restore(pool: np.ndarray, plane_stride: int, block_stride: int, n_planes: int, n_blocks: int,
               block_bytes: int, image: np.ndarray, img_plane_stride: int, img_slot_stride: int, ids: np.ndarray):
    """Scatter selected slots into the host pool (modified in place).

    Returns (status, block_digests, kv_digests, skipped).
    """
    pool_b = pool.view(np.uint8).reshape(-1)
    img = _bytes_view(image)
    ids = np.ascontiguousarray(ids, dtype=np.int32)
    k = block_bytes // BLOCK
    bd = np.zeros(len(ids) * n_planes * k, dtype=np.uint64)
    kd = np.zeros(len(ids), dtype=np.uint64)
    skipped = C.c_uint64(0)
    rc = lib().gmso_kv_restore(_ptr(pool_b), plane_stride, block_stride, n_planes, n_blocks, block_bytes, _ptr(img),
                               img_plane_stride, img_slot_stride, _ptr(ids), len(ids), _ptr(bd), _ptr(kd),
                               C.addressof(skipped))
    return int(rc), bd, kd, int(skipped.value)


def kv_capture(pool: np.ndarray, plane_stride: int, block_stride: int, n_planes: int, n_blocks: int,
               block_bytes: int, image: np.ndarray, img_plane_stride: int, img_slot_stride: int, ids: np.ndarray):
    """Gather selected pool blocks into the host image (modified in place).

    Returns (status, block_digests, kv_digests, skipped).
    """
    pool_b = _bytes_view(pool)
    img = image.view(np.uint8).reshape(-1)
    ids = np.ascontiguousarray(ids, dtype=np.int32)
    k = block_bytes // BLOCK
    bd = np.zeros(len(ids) * n_planes * k, dtype=np.uint64)
    kd = np.zeros(len(ids), dtype=np.uint64)
    skipped = C.c_uint64(0)
    rc = lib().gmso_kv_capture(_ptr(pool_b), plane_stride, block_stride, n_planes, n_blocks, block_bytes, _ptr(img),
                               img_plane_stride, img_slot_stride, _ptr(ids), len(ids), _ptr(bd), _ptr(kd),
                               C.addressof(skipped))
    return int(rc), bd, kd, int(skipped.value)


def kv_digest(pool: np.ndarray, plane_stride: int, block_stride: int, n_planes: int, n_blocks: int,
              block_bytes: int, ids: np.ndarray):
    """Digest selected pool blocks where they lie (the pool is only read).

    Returns (status, block_digests, kv_digests, skipped).
    """
    pool_b = _bytes_view(pool)
    ids = np.ascontiguousarray(ids, dtype=np.int32)
    k = block_bytes // BLOCK
    bd = np.zeros(len(ids) * n_planes * k, dtype=np.uint64)
    kd = np.zeros(len(ids), dtype=np.uint64)
    skipped = C.c_uint64(0)
    rc = lib().gmso_kv_digest(_ptr(pool_b), plane_stride, block_stride, n_planes, n_blocks, block_bytes, _ptr(ids),
                              len(ids), _ptr(bd), _ptr(kd), C.addressof(skipped))
    return int(rc), bd, kd, int(skipped.value)


def kv_verify(n_planes: int, n_blocks: int, block_bytes: int, ids: np.ndarray, computed: np.ndarray, expected: np.ndarray,
              cap: int):
    """Differing (block_id, plane, sub_block, list_pos) records in (list position, plane, sub-block) order.

    Returns (count, records[:min(count, cap)]).
    """
    ids = np.ascontiguousarray(ids, dtype=np.int32)
    computed = np.ascontiguousarray(computed, dtype=np.uint64)
    expected = np.ascontiguousarray(expected, dtype=np.uint64)
    assert computed.size == expected.size == len(ids) * n_planes * (block_bytes // BLOCK)
    out = np.zeros(max(cap, 1), dtype=KV_MISMATCH_DTYPE)
    n = int(lib().gmso_kv_verify(n_planes, n_blocks, block_bytes, _ptr(ids), len(ids), _ptr(computed), _ptr(expected),
                                 _ptr(out), int(cap)))
    return n, out[: min(n, cap)].copy()
