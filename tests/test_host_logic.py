"""CPU-only checks of the C-ABI library: it loads without a GPU, exports every symbol the
header declares, and its host logic (validation, block layout, work-list construction) agrees
with the oracle's validation and with the invariants of a partition.  No kernel is launched."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2609_25451_b200 import build as gms_build
from paper_2609_25451_b200 import gms
from paper_2609_25451_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
FAKE_BASE = 0x7F0000000000  # stands in for a device slab; never dereferenced in host-only mode


@pytest.fixture(scope="module", autouse=True)
def built():
    gms_build.build()


def entries_of(w, base=FAKE_BASE):
    return gms.make_entries((r["tensor_id"], r["src_offset"], base + int(r["dst_offset"]), r["nbytes"]) for r in w.rows)


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "gms.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(gms_[a-z0-9_]+)\s*\(", header))
    assert declared == set(gms.EXPORTS)
    L = ctypes.CDLL(gms.LIB_PATH)
    for name in declared:
        assert hasattr(L, name), name
    assert gms.gms_version() == 0x00010000
    assert gms.gms_strerror(gms.ERR_OVERLAP).startswith("destination")


def test_struct_sizes_match_the_header():
    assert gms.ENTRY_DTYPE.itemsize == 32 and gms.MISMATCH_DTYPE.itemsize == 16
    assert ctypes.sizeof(gms.KvPool) == 40


def test_validation_matches_oracle_status(oracle):
    cases = [
        ([(1, 0, 0, 100), (2, 112, 112, 100)], oracle.OK),
        ([(1, 8, 0, 100)], oracle.ERR_ALIGN),
        ([(1, 0, 8, 100)], oracle.ERR_ALIGN),
        ([(1, 992, 0, 16)], oracle.ERR_RANGE),
        ([(1, 0, 0, 2**64 - 1)], oracle.ERR_RANGE),
        ([(1, 0, 0, 100), (2, 112, 96, 100)], oracle.ERR_OVERLAP),
        ([(1, 0, 0, 100), (1, 112, 112, 100)], oracle.ERR_DUP_ID),
        ([(1, 0, 0, 100), (2, 0, 112, 100), (3, 0, 0, 0)], oracle.OK),
        ([], oracle.OK),
    ]
    for rows, want in cases:
        assert oracle.validate(oracle.make_record(rows), 1000, 1 << 40) == want
        ent = gms.make_entries((a, b, FAKE_BASE + c, d) for a, b, c, d in rows)
        if want == oracle.OK:
            m = gms.gms_manifest_build(ent, 1000, gms.BUILD_HOST_ONLY)
            assert m.n_tensors == len(rows)
            m.close()
        else:
            with pytest.raises(gms.GmsError) as ei:
                gms.gms_manifest_build(ent, 1000, gms.BUILD_HOST_ONLY)
            assert ei.value.status == want  # the library's codes are the oracle's, by value


def test_random_invalid_records_agree_with_oracle(oracle):
    rng = np.random.default_rng(99)
    agree = 0
    for _ in range(300):
        n = int(rng.integers(1, 6))
        rows = [(int(rng.integers(0, 4)), int(rng.integers(0, 40)) * 8, int(rng.integers(0, 40)) * 8,
                 int(rng.integers(0, 200))) for _ in range(n)]
        want = oracle.validate(oracle.make_record(rows), 256, 1 << 40)
        ent = gms.make_entries((a, b, FAKE_BASE + c, d) for a, b, c, d in rows)
        try:
            gms.gms_manifest_build(ent, 256, gms.BUILD_HOST_ONLY).close()
            got = 0
        except gms.GmsError as e:
            got = e.status
        # several defects can coexist and the two sides may name different ones; accept/reject must agree
        assert (got == 0) == (want == 0)
        agree += got == want
    assert agree > 150


def test_validation_of_thousands_of_tensors_agrees_with_the_oracle(oracle):
    """From 2,048 tensors on the library's validation sorts its keys with a radix sort; the oracle's quadratic check
    of the same records must reach the same verdict -- for a clean record, one duplicated id, one pair of overlapping
    destinations far apart in the list, and sources that overlap (legal)."""
    w = W.pack_layout("many", [int(x) for x in np.random.default_rng(5).integers(0, 3000, 5000)], seed=8)
    base_rows = [(int(r["tensor_id"]), int(r["src_offset"]), int(r["dst_offset"]), int(r["nbytes"])) for r in w.rows]
    live = [i for i, r in enumerate(base_rows) if r[3] > 64]

    def verdicts(rows):
        want = oracle.validate(oracle.make_record(rows), w.image_bytes, 1 << 40)
        ent = gms.make_entries((a, b, FAKE_BASE + c, d) for a, b, c, d in rows)
        try:
            m = gms.gms_manifest_build(ent, w.image_bytes, gms.BUILD_HOST_ONLY)
            n_chunks = gms.gms_manifest_chunk_count(m)
            covered = sum(gms.gms_manifest_chunk(m, i)[2] for i in range(0, n_chunks, 97))  # the lists still build
            assert covered > 0
            m.close()
            return want, 0
        except gms.GmsError as e:
            return want, e.status

    assert verdicts(base_rows) == (oracle.OK, 0)
    dup = list(base_rows)
    dup[4321] = (dup[17][0],) + dup[4321][1:]
    assert verdicts(dup) == (oracle.ERR_DUP_ID, gms.ERR_DUP_ID)
    ovl = list(base_rows)
    i, j = live[3], live[-5]
    ovl[j] = (ovl[j][0], ovl[j][1], ovl[i][2] + 16, ovl[j][3])  # destination j now starts inside destination i
    assert verdicts(ovl) == (oracle.ERR_OVERLAP, gms.ERR_OVERLAP)
    shared = list(base_rows)
    shared[j] = (shared[j][0], shared[i][1], shared[j][2], min(shared[j][3], shared[i][3]))  # same source bytes: legal
    assert verdicts(shared) == (oracle.OK, 0)


def test_index_limits_are_refused_before_anything_is_built():
    # digest slots are 32-bit on the device: 2^32 - 1 blocks or more (16 TiB of payload) is refused during validation
    big = 4096 * (2**32 - 1)
    ent = gms.make_entries([(1, 0, FAKE_BASE, big)])
    with pytest.raises(gms.GmsError) as ei:
        gms.gms_manifest_build(ent, big, gms.BUILD_HOST_ONLY)
    assert ei.value.status == gms.ERR_RANGE
    # the same limit reached by the sum over two tensors
    half = 4096 * 2**31
    ent = gms.make_entries([(1, 0, FAKE_BASE, half), (2, half, FAKE_BASE + half, half)])
    with pytest.raises(gms.GmsError) as ei:
        gms.gms_manifest_build(ent, 2 * half, gms.BUILD_HOST_ONLY)
    assert ei.value.status == gms.ERR_RANGE
    # a destination range that wraps the address space
    ent = gms.make_entries([(1, 0, 2**64 - 4096, 8192)])
    with pytest.raises(gms.GmsError) as ei:
        gms.gms_manifest_build(ent, 8192, gms.BUILD_HOST_ONLY)
    assert ei.value.status == gms.ERR_RANGE
    # a byte range of 100 GB in one tensor is fine on the host (25 M blocks, 6 M chunks)
    n = 100 * 10**9
    m = gms.gms_manifest_build(gms.make_entries([(1, 0, FAKE_BASE, n)]), n, gms.BUILD_HOST_ONLY)
    assert m.n_blocks == (n + 4095) // 4096 and gms.gms_manifest_chunk_count(m) == (m.n_blocks + 3) // 4
    m.close()


def test_null_and_flag_errors():
    out = ctypes.c_void_p()
    assert gms.lib().gms_manifest_build(None, 3, 100, 0, ctypes.byref(out)) == gms.ERR_NULL
    assert gms.lib().gms_manifest_build(None, 0, 100, 0, None) == gms.ERR_NULL
    assert gms.lib().gms_manifest_build(None, 0, 100, 0x80, ctypes.byref(out)) == gms.ERR_ARG
    assert gms.lib().gms_manifest_info(None, None, None, None) == gms.ERR_NULL
    assert gms.lib().gms_manifest_destroy(None) == gms.OK


@pytest.mark.parametrize("make", [
    lambda: W.tiny_manifest(),
    lambda: W.mixed_manifest(n_small=500, n_large=2, large_bytes=3 << 20, round16=False),
    lambda: W.llama3_8b_manifest(shrink=16),
    lambda: W.pack_layout("edge", [0, 1, 15, 16, 17, 4095, 4096, 4097, 8191, 8192, 8193, 0, 131072, 131073, 300000], seed=4),
])
def test_block_layout_and_chunks_partition_every_tensor(oracle, make):
    w = make()
    m = gms.gms_manifest_build(entries_of(w), w.image_bytes, gms.BUILD_HOST_ONLY)
    rec = oracle.make_record((r["tensor_id"], r["src_offset"], r["dst_offset"], r["nbytes"]) for r in w.rows)
    base, total = oracle.block_bases(rec)
    assert (m.n_tensors, m.n_blocks, m.payload_bytes) == (len(w.rows), total, w.payload_bytes)
    for t in range(len(w.rows)):
        assert gms.gms_manifest_block_base(m, t) == int(base[t])
    covered = {}
    prev = None
    for i in range(gms.gms_manifest_chunk_count(m)):
        t, off, nb = gms.gms_manifest_chunk(m, i)
        assert 1 <= nb <= 32 * 4096 and off % 4096 == 0
        assert nb % 4096 == 0 or off + nb == int(w.rows[t]["nbytes"])  # only a tensor's last chunk is ragged
        covered.setdefault(t, []).append((off, nb))
        assert prev is None or nb <= prev  # large chunks are claimed first
        prev = nb
    for t, r in enumerate(w.rows):
        runs = sorted(covered.get(t, []))
        pos = 0
        for off, nb in runs:
            assert off == pos
            pos += nb
        assert pos == int(r["nbytes"])
    # a host-only manifest refuses device work instead of computing anything on the CPU
    assert gms.lib().gms_digest(m.handle, None, None, None) == gms.ERR_STATE
    assert gms.lib().gms_restore(m.handle, ctypes.c_void_p(16), 0, None, None, None) == gms.ERR_STATE
    m.close()


def test_kv_argument_checks_need_no_gpu():
    pool = gms.KvPool(base=FAKE_BASE, plane_stride=1 << 20, block_stride=32768, n_planes=2, n_blocks=8, block_bytes=32768)
    st = ctypes.c_void_p(FAKE_BASE)
    call = lambda p, kind=0, ips=1 << 20, iss=32768: gms.lib().gms_kv_restore(
        ctypes.byref(p), ctypes.c_void_p(FAKE_BASE), ips, iss, kind, ctypes.c_void_p(FAKE_BASE), 4, None, None, st, None)
    bad = gms.KvPool(base=FAKE_BASE, plane_stride=1 << 20, block_stride=32768, n_planes=2, n_blocks=8, block_bytes=1000)
    assert call(bad) == gms.ERR_ALIGN
    big = gms.KvPool(base=FAKE_BASE, plane_stride=1 << 20, block_stride=1 << 18, n_planes=2, n_blocks=4, block_bytes=1 << 18)
    assert call(big) == gms.ERR_ARG
    assert call(pool, kind=7) == gms.ERR_KIND
    assert call(pool, iss=32760) == gms.ERR_ALIGN
    assert gms.lib().gms_kv_restore(None, None, 0, 0, 0, None, 0, None, None, st, None) == gms.ERR_NULL
    # planes that would share bytes: a plane spans (n_blocks - 1) * block_stride + block_bytes
    span = 7 * 32768 + 32768
    tight = gms.KvPool(base=FAKE_BASE, plane_stride=span - 16, block_stride=32768, n_planes=2, n_blocks=8, block_bytes=32768)
    assert call(tight) == gms.ERR_ARG
    assert gms.lib().gms_kv_digest(ctypes.byref(tight), ctypes.c_void_p(FAKE_BASE), 4, None, None, st, None) == gms.ERR_ARG
    one_plane = gms.KvPool(base=FAKE_BASE, plane_stride=0, block_stride=32768, n_planes=1, n_blocks=8, block_bytes=32768)
    assert call(one_plane, kind=7) == gms.ERR_KIND  # a single plane has no neighbour to overlap: the check is passed
    # gms_kv_verify: host-side checks
    kvv = lambda p, n_sel=4, ids=FAKE_BASE, cap=4: gms.lib().gms_kv_verify(
        ctypes.byref(p), ctypes.c_void_p(ids), n_sel, ctypes.c_void_p(FAKE_BASE), ctypes.c_void_p(FAKE_BASE),
        ctypes.c_void_p(FAKE_BASE), cap, st, None, None)
    assert kvv(bad) == gms.ERR_ALIGN and kvv(big) == gms.ERR_ARG
    assert kvv(pool) == gms.ERR_NULL  # slots to compare but no scratch
    assert gms.kv_verify_scratch_words(0) == 1 and gms.kv_verify_scratch_words(2048) == 2 and gms.kv_verify_scratch_words(2049) == 3


def test_workload_recipes_have_the_stated_sizes():
    w = W.llama3_8b_manifest()
    assert len(w.rows) == 291 and w.payload_bytes == 16_060_522_496 and w.n_blocks == 3_921_026
    s = W.llama3_70b_tp8_shard_manifest()
    assert len(s.rows) == 722 and s.payload_bytes == 17_640_718_336
    s2 = W.llama3_70b_tp8_shard_manifest(image_bytes=32 << 30)
    assert s2.payload_bytes <= 32 << 30 and len(s2.rows) > 722
    k = W.kv_pool_workload()
    assert (k.n_planes, k.n_blocks, k.block_bytes, len(k.ids)) == (64, 28610, 32768, 2861)
    assert len(set(k.ids.tolist())) == len(k.ids) and k.pool_bytes == 59_999_518_720
    mx = W.mixed_manifest()
    assert len(mx.rows) == 10008 and (mx.rows["nbytes"] % 16 == 0).all()
    t = W.tiny_manifest()
    assert len(t.rows) == 64 and t.rows["nbytes"].min() >= 4096 and t.rows["nbytes"].max() <= 1 << 20
    # destinations never overlap and keep their guard bands
    for wl in (t, mx):
        o = np.argsort(wl.rows["dst_offset"])
        ends = wl.rows["dst_offset"][o] + wl.rows["nbytes"][o]
        assert (wl.rows["dst_offset"][o][1:] >= ends[:-1] + W.GUARD - 15).all()
