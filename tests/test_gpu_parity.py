"""GPU parity: the CUDA library, called through the C ABI, against the CPU oracle on the same
seeded inputs -- element by element, bit-exact (everything here is integer work): destination
bytes, block digests, tensor digests, mismatch lists and counts, KV status counts.  Sizes are
small enough for the oracle yet span many chunks, several ring slots per warp and ragged tails.
Guard bands around every destination and canary words around every output array catch stray writes."""
import ctypes
import zlib

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

from paper_2609_25451_b200 import gms  # noqa: E402
from paper_2609_25451_b200 import workloads as W  # noqa: E402

from gpu_harness import CANARY, FILL, PAD, DeviceWorkload, guarded_u64, oracle_record, payload_of  # noqa: E402

EDGE_SIZES = [0, 1, 7, 8, 9, 15, 16, 17, 31, 4080, 4095, 4096, 4097, 4111, 4112, 8191, 8192, 8193, 0, 12288,
              65535, 65536, 65537, 131071, 131072, 131073, 262144 + 5, 1 << 20, (1 << 20) + 4097, 3, 0]

WORKLOADS = {
    "tiny64": lambda: W.tiny_manifest(),
    "edge": lambda: W.pack_layout("edge", EDGE_SIZES, seed=11),
    "mixed-odd": lambda: W.mixed_manifest(n_small=3000, n_large=2, large_bytes=(8 << 20) + 24, round16=False),
    "llama8b/16": lambda: W.llama3_8b_manifest(shrink=16),
}


def oracle_restore(oracle, w, image):
    slab = np.full(w.slab_bytes, FILL, np.uint8)
    rc, bd, td = oracle.restore(oracle_record(oracle, w), image, slab)
    assert rc == 0
    return slab, bd, td


@pytest.mark.parametrize("name", sorted(WORKLOADS))
def test_restore_digest_verify_parity(oracle, name):
    w = WORKLOADS[name]()
    image = W.random_bytes_host(w.image_bytes, seed=zlib.crc32(name.encode()) & 0xFFFF)
    want_slab, want_bd, want_td = oracle_restore(oracle, w, image)
    d = DeviceWorkload(w, image)

    bd, td = d.restore()
    got_slab = d.slab_host()
    assert np.array_equal(got_slab, want_slab), "destination bytes (or guard bands) differ"
    assert np.array_equal(bd, want_bd) and np.array_equal(td, want_td)

    # digest in place: same digests, destinations untouched
    bd2, td2 = d.digest()
    assert np.array_equal(bd2, want_bd) and np.array_equal(td2, want_td)
    assert np.array_equal(d.slab_host(), want_slab)

    # record the digests; a clean verify reports nothing
    gms.gms_manifest_set_expected(d.m, d.bd_ptr())
    assert d.verify(cap=8) == (0, [])

    # host-made single-bit flips are named exactly, in (entry, block) order
    flips = W.flip_positions(w, 3, seed=5)
    rec = oracle_record(oracle, w)
    for row, byte, bit in flips:
        d.flip(row, byte, bit)
        want_slab[int(w.rows[row]["dst_offset"]) + byte] ^= 1 << bit
    bd3, td3 = d.digest()
    _, obd3, otd3 = oracle.digest(rec, want_slab)
    assert np.array_equal(bd3, obd3) and np.array_equal(td3, otd3)
    count, pairs = d.verify(cap=8)
    ocount, omm = oracle.verify(rec, obd3, want_bd, cap=8)
    assert count == ocount == 3
    assert pairs == [(int(m["tensor_id"]), int(m["block"])) for m in omm]
    assert sorted(pairs) == sorted((int(w.rows[r]["tensor_id"]), b // 4096) for r, b, _ in flips)
    # cap smaller than the count: total still reported, only cap entries written
    count, pairs = d.verify(cap=2)
    assert count == 3 and pairs == [(int(m["tensor_id"]), int(m["block"])) for m in omm][:2]
    count, pairs = d.verify(cap=0)
    assert count == 3 and pairs == []
    # the fused calls: same digests, same list, same count as the oracle's digest + verify
    want_pairs = [(int(m["tensor_id"]), int(m["block"])) for m in omm]
    for cap in (8, 2, 0):
        fbd, ftd, count, pairs = d.fused(cap)
        assert np.array_equal(fbd, obd3) and np.array_equal(ftd, otd3)
        assert count == 3 and pairs == want_pairs[:cap]
    assert np.array_equal(d.slab_host(), want_slab)
    # restore + verify in one pass: the flips are overwritten, nothing differs any more
    clean_slab, _, _ = oracle_restore(oracle, w, image)
    fbd, ftd, count, pairs = d.fused(8, restore=True)
    assert np.array_equal(fbd, want_bd) and np.array_equal(ftd, want_td) and (count, pairs) == (0, [])
    assert np.array_equal(d.slab_host(), clean_slab)
    d.close()


def test_optional_outputs_may_be_null(oracle):
    w = W.pack_layout("opt", [5000, 70000, 16, 0, 4096], seed=3)
    image = W.random_bytes_host(w.image_bytes, seed=8)
    want_slab, want_bd, want_td = oracle_restore(oracle, w, image)
    d = DeviceWorkload(w, image)
    for want_b, want_t in ((True, False), (False, True), (False, False)):
        d.slab.fill_(FILL)
        bd, td = d.restore(want_bd=want_b, want_td=want_t)
        assert np.array_equal(d.slab_host(), want_slab)
        assert np.array_equal(bd, want_bd) if want_b else (bd == CANARY).all()
        assert np.array_equal(td, want_td) if want_t else (td == CANARY).all()
    d.close()


def test_empty_manifests(oracle):
    for sizes in ([], [0, 0, 0]):
        w = W.pack_layout("empty", sizes, seed=1)
        d = DeviceWorkload(w, np.zeros(w.image_bytes, np.uint8))
        bd, td = d.restore()
        assert bd.size == 0 and (td == 0).all() and td.size == len(sizes)
        bd, td = d.digest()
        assert (td == 0).all()
        gms.gms_manifest_set_expected(d.m, d.bd_ptr())
        assert d.verify(cap=4) == (0, [])
        assert d.fused(4)[2:] == (0, []) and d.fused(4, restore=True)[2:] == (0, [])
        assert (d.slab_host() == FILL).all()
        d.close()


def test_results_do_not_depend_on_entry_order_or_chunking(oracle, monkeypatch):
    w = W.mixed_manifest(n_small=800, n_large=1, large_bytes=5 << 20, round16=False, seed=77)
    image = W.random_bytes_host(w.image_bytes, seed=9)
    d = DeviceWorkload(w, image)
    bd, td = d.restore()
    slab = d.slab_host()
    by_id = {int(r["tensor_id"]): int(td[t]) for t, r in enumerate(w.rows)}
    d.close()
    # permuted entries: per-id results unchanged, destination bytes identical
    perm = np.random.default_rng(5).permutation(len(w.rows))
    w2 = W.Workload(w.name, w.rows[perm].copy(), w.image_bytes, w.slab_bytes)
    d2 = DeviceWorkload(w2, image)
    bd2, td2 = d2.restore()
    assert np.array_equal(d2.slab_host(), slab)
    assert {int(r["tensor_id"]): int(td2[t]) for t, r in enumerate(w2.rows)} == by_id
    d2.close()
    # different internal chunk length: every output bit-identical
    monkeypatch.setenv("GMS_TUNING_HOOKS", "1")
    for blocks, digest_blocks in (("1", "32"), ("5", "3"), ("32", "1")):
        monkeypatch.setenv("GMS_CHUNK_BLOCKS", blocks)
        monkeypatch.setenv("GMS_CHUNK_BLOCKS_DIGEST", digest_blocks)
        d3 = DeviceWorkload(w, image)
        assert gms.gms_manifest_chunk(d3.m, 0)[2] == min(int(blocks) * 4096, int(w.rows["nbytes"].max()))
        bd3, td3 = d3.restore()
        assert np.array_equal(bd3, bd) and np.array_equal(td3, td) and np.array_equal(d3.slab_host(), slab)
        bd4, td4 = d3.digest()
        assert np.array_equal(bd4, bd) and np.array_equal(td4, td)
        d3.close()
    # without the master switch the hooks are ignored
    monkeypatch.delenv("GMS_TUNING_HOOKS")
    monkeypatch.setenv("GMS_CHUNK_BLOCKS", "1")
    d4 = DeviceWorkload(w, image)
    assert gms.gms_manifest_chunk(d4.m, 0)[2] > 4096
    d4.close()


@pytest.mark.parametrize("scale", [1, 8])  # 8.7 K blocks: single-CTA verify; 70 K blocks: count / scan / emit
def test_many_mismatches_exceed_cap_in_order(oracle, scale):
    w = W.pack_layout("many", [4096 * 700 * scale + 100, 4096 * 3000 * scale, 10, 4096 * 5000 * scale + 1], seed=2)
    image = W.random_bytes_host(w.image_bytes, seed=10)
    rec = oracle_record(oracle, w)
    d = DeviceWorkload(w, image)
    want_slab, want_bd, _ = oracle_restore(oracle, w, image)
    d.restore()
    gms.gms_manifest_set_expected(d.m, d.bd_ptr())
    # corrupt every 3rd block of the slab region wholesale (host-made corruption)
    rng = np.random.default_rng(4)
    for row in range(len(w.rows)):
        nb = int(w.rows[row]["nbytes"])
        for b in range(0, (nb + 4095) // 4096, 3):
            pos = int(w.rows[row]["dst_offset"]) + min(nb - 1, b * 4096 + int(rng.integers(0, 4096)))
            want_slab[pos] ^= 0x10
    d.slab.copy_(torch.from_numpy(want_slab))
    bd, _ = d.digest()
    _, obd, _ = oracle.digest(rec, want_slab)
    assert np.array_equal(bd, obd)
    for cap in (100, 5000):
        count, pairs = d.verify(cap=cap)
        ocount, omm = oracle.verify(rec, obd, want_bd, cap=cap)
        assert count == ocount and count > 2500
        assert pairs == [(int(m["tensor_id"]), int(m["block"])) for m in omm]
        fbd, _, fcount, fpairs = d.fused(cap)  # the compare folded into the digest pass
        assert np.array_equal(fbd, obd) and fcount == ocount and fpairs == pairs
    # restore + verify against digests recorded from the damaged state: every block that was damaged now differs
    gms.gms_manifest_set_expected(d.m, d.bd_ptr())
    fbd, _, fcount, fpairs = d.fused(5000, restore=True)
    ocount2, omm2 = oracle.verify(rec, want_bd, obd, cap=5000)
    assert np.array_equal(fbd, want_bd) and fcount == ocount2 == ocount
    assert fpairs == [(int(m["tensor_id"]), int(m["block"])) for m in omm2]
    d.slab.copy_(torch.from_numpy(want_slab))
    gms.gms_manifest_set_expected(d.m, torch.from_numpy(want_bd.view(np.int64)).cuda())
    bd, _ = d.digest()
    # the computed digests may sit at an address that is only 8-byte aligned
    shifted = torch.zeros(d.nb + 1, dtype=torch.int64, device="cuda")
    shifted[1:] = d.bd[PAD:PAD + d.nb]
    out = torch.zeros(2 * 16, dtype=torch.int64, device="cuda")
    cnt = torch.zeros(1, dtype=torch.int64, device="cuda")
    gms.gms_verify(d.m, shifted.data_ptr() + 8, out, 16, cnt)
    torch.cuda.synchronize()
    ocount, omm = oracle.verify(rec, obd, want_bd, cap=16)
    assert int(cnt.item()) == ocount
    assert out.cpu().numpy().view(np.uint64).reshape(16, 2).tolist() == [[int(m["tensor_id"]), int(m["block"])] for m in omm]
    # per-tensor summary = the oracle's full mismatch list counted per tensor id (entry order)
    ocount, omm = oracle.verify(rec, obd, want_bd, cap=1 << 20)
    want_counts = [sum(1 for m in omm if int(m["tensor_id"]) == int(r["tensor_id"])) for r in w.rows]
    tc = torch.full((len(w.rows) + 2,), 0x7777, dtype=torch.int32, device="cuda")
    gms.gms_verify_tensors(d.m, d.bd_ptr(), tc.data_ptr() + 4)
    torch.cuda.synchronize()
    got = tc.cpu().tolist()
    assert got[0] == 0x7777 and got[-1] == 0x7777 and got[1:-1] == want_counts and sum(want_counts) == ocount
    d.close()


def test_host_mapped_source_parity(oracle):
    w = W.mixed_manifest(n_small=400, n_large=1, large_bytes=(2 << 20) + 40, round16=False, seed=31)
    image = W.random_bytes_host(w.image_bytes, seed=12)
    want_slab, want_bd, want_td = oracle_restore(oracle, w, image)
    hptr, dview, arr = gms.gms_host_image_alloc(w.image_bytes)
    try:
        arr[:] = image
        d = DeviceWorkload(w, image)
        bd, td = d.restore(image=dview, kind=gms.SRC_HOST_MAPPED)
        assert np.array_equal(d.slab_host(), want_slab)
        assert np.array_equal(bd, want_bd) and np.array_equal(td, want_td)
        # the fused restore + verify reads the mapped image just the same
        gms.gms_manifest_set_expected(d.m, d.bd_ptr())
        d.slab.fill_(FILL)
        d.reset_outputs()
        out = torch.full((2 * 4,), -1, dtype=torch.int64, device="cuda")
        cnt = torch.full((1,), -1, dtype=torch.int64, device="cuda")
        gms.gms_restore_verify(d.m, dview, gms.SRC_HOST_MAPPED, d.bd_ptr(), d.td_ptr(), out, 4, cnt)
        torch.cuda.synchronize()
        assert int(cnt.item()) == 0 and (out == -1).all() and np.array_equal(d.slab_host(), want_slab)
        assert np.array_equal(payload_of(d.bd, d.nb), want_bd) and np.array_equal(payload_of(d.td, d.nt), want_td)
        with pytest.raises(gms.GmsError) as ei:
            gms.gms_restore_verify(d.m, dview, gms.SRC_DEVICE, d.bd_ptr(), d.td_ptr(), out, 4, cnt)
        assert ei.value.status == gms.ERR_KIND
        with pytest.raises(gms.GmsError) as ei:
            gms.gms_restore_verify(d.m, dview, gms.SRC_HOST_MAPPED, None, d.td_ptr(), out, 4, cnt)
        assert ei.value.status == gms.ERR_NULL
        # the pointer must be what image_kind says
        with pytest.raises(gms.GmsError) as ei:
            gms.gms_restore(d.m, dview, gms.SRC_DEVICE, None, None)
        assert ei.value.status == gms.ERR_KIND
        with pytest.raises(gms.GmsError) as ei:
            gms.gms_restore(d.m, d.image, gms.SRC_HOST_MAPPED, None, None)
        assert ei.value.status == gms.ERR_KIND
        with pytest.raises(gms.GmsError) as ei:
            gms.gms_restore(d.m, d.image.data_ptr() + 8, gms.SRC_DEVICE, None, None)
        assert ei.value.status == gms.ERR_ALIGN
        d.close()
    finally:
        torch.cuda.synchronize()
        gms.gms_host_image_free(hptr)


def run_kv(oracle, n_planes, n_blocks, block_bytes, ids, plane_gap, seed, host_mapped=False):
    k = block_bytes // 4096
    plane_stride = n_blocks * block_bytes + plane_gap
    n_sel = len(ids)
    ips, iss = max(n_sel, 1) * block_bytes + 64, block_bytes
    pool_h = W.random_bytes_host(n_planes * plane_stride, seed)
    img_h = W.random_bytes_host(n_planes * ips, seed + 1)
    want_pool = pool_h.copy()
    rc, obd, okd, oskip = oracle.kv_restore(want_pool, plane_stride, block_bytes, n_planes, n_blocks, block_bytes, img_h,
                                            ips, iss, ids)
    assert rc == 0
    pool = torch.from_numpy(pool_h).cuda()
    hptr = None
    if host_mapped:
        hptr, img_ptr, arr = gms.gms_host_image_alloc(img_h.size)
        arr[:] = img_h
    else:
        img = torch.from_numpy(img_h).cuda()
        img_ptr = img.data_ptr()
    ids_d = torch.from_numpy(np.ascontiguousarray(ids, dtype=np.int32)).cuda()
    bd, kd, st = guarded_u64(n_sel * n_planes * k), guarded_u64(n_sel), guarded_u64(4)
    desc = gms.KvPool(base=pool.data_ptr(), plane_stride=plane_stride, block_stride=block_bytes, n_planes=n_planes,
                      n_blocks=n_blocks, block_bytes=block_bytes)
    gms.gms_kv_restore(desc, img_ptr, ips, iss, gms.SRC_HOST_MAPPED if host_mapped else gms.SRC_DEVICE, ids_d, n_sel,
                       bd.data_ptr() + 8 * PAD, kd.data_ptr() + 8 * PAD, st.data_ptr() + 8 * PAD)
    torch.cuda.synchronize()
    status = payload_of(st, 4)
    assert int(status[0]) == oskip and int(status[1]) == 0
    assert np.array_equal(pool.cpu().numpy(), want_pool), "pool bytes differ"
    assert np.array_equal(payload_of(bd, n_sel * n_planes * k), obd)
    assert np.array_equal(payload_of(kd, n_sel), okd)
    if hptr:
        gms.gms_host_image_free(hptr)


def test_kv_restore_parity(oracle):
    rng = np.random.default_rng(41)
    ids = rng.permutation(300)[:90].astype(np.int32)
    run_kv(oracle, n_planes=6, n_blocks=300, block_bytes=32768, ids=ids, plane_gap=4096, seed=50)


def test_kv_restore_out_of_range_ids_are_skipped_and_counted(oracle):
    ids = np.array([5, -1, 0, 40, 39, 2**31 - 1, -(2**31), 7], np.int32)
    run_kv(oracle, n_planes=4, n_blocks=40, block_bytes=8192, ids=ids, plane_gap=0, seed=60)


def test_kv_restore_other_block_sizes_and_host_source(oracle):
    rng = np.random.default_rng(43)
    run_kv(oracle, 3, 64, 4096, rng.permutation(64)[:20].astype(np.int32), 256, 70)
    run_kv(oracle, 2, 16, 131072, rng.permutation(16)[:9].astype(np.int32), 0, 80)
    run_kv(oracle, 5, 50, 32768, rng.permutation(50)[:11].astype(np.int32), 512, 90, host_mapped=True)
    run_kv(oracle, 5, 50, 32768, np.zeros(0, np.int32), 0, 95)


def test_device_written_work_lists_equal_the_hosts(monkeypatch):
    """gms_manifest_build writes the chunk records on the device; with the check hook on it reads them back and
    compares them with the host's construction of the same order (a difference would make the build fail).  The
    introspection calls, which use the host's lists, must describe a partition of every tensor."""
    monkeypatch.setenv("GMS_TUNING_HOOKS", "1")
    monkeypatch.setenv("GMS_CHECK_TABLES", "1")
    for w in (W.pack_layout("edge", EDGE_SIZES, seed=11), W.mixed_manifest(n_small=3000, n_large=2, large_bytes=(8 << 20) + 24, round16=False),
              W.llama3_8b_manifest(shrink=8), W.pack_layout("empty", [0, 0], seed=1)):
        for blocks in ("1", "4", "7", "32"):
            monkeypatch.setenv("GMS_CHUNK_BLOCKS", blocks)
            monkeypatch.setenv("GMS_CHUNK_BLOCKS_DIGEST", str(33 - int(blocks)))
            d = DeviceWorkload(w, np.zeros(w.image_bytes, np.uint8))  # the build itself is the check
            covered = {}
            for i in range(gms.gms_manifest_chunk_count(d.m)):
                t, off, n = gms.gms_manifest_chunk(d.m, i)
                covered.setdefault(t, []).append((off, n))
            for t, r in enumerate(w.rows):
                pieces = sorted(covered.get(t, []))
                assert sum(n for _, n in pieces) == int(r["nbytes"])
                assert all(pieces[k][0] + pieces[k][1] == pieces[k + 1][0] for k in range(len(pieces) - 1))
            d.close()


def test_thirty_thousand_small_tensors_and_exact_chunk_multiples(oracle):
    """Many tensors, most of them shorter than one chunk (so nearly every chunk is some tensor's short last one and
    the list order is decided by the ranking of those), next to tensors that are exact multiples of the chunk
    lengths (no short chunk at all) and empty ones: bytes, digests, fused verify against the oracle."""
    rng = np.random.default_rng(123)
    sizes = [int(x) for x in rng.integers(0, 9000, 30000)]
    sizes[::97] = [0] * len(sizes[::97])
    sizes += [16384 * 3, 32768 * 5, 16384, 32768, 4096, 65536 * 7]
    w = W.pack_layout("many-small", sizes, seed=31, guard=16)
    image = W.random_bytes_host(w.image_bytes, seed=32)
    want_slab, want_bd, want_td = oracle_restore(oracle, w, image)
    d = DeviceWorkload(w, image)
    bd, td = d.restore()
    assert np.array_equal(d.slab_host(), want_slab) and np.array_equal(bd, want_bd) and np.array_equal(td, want_td)
    bd2, td2 = d.digest()
    assert np.array_equal(bd2, want_bd) and np.array_equal(td2, want_td)
    gms.gms_manifest_set_expected(d.m, d.bd_ptr())
    rec = oracle_record(oracle, w)
    flips = W.flip_positions(w, 40, seed=33)
    for row, byte, bit in flips:
        d.flip(row, byte, bit)
        want_slab[int(w.rows[row]["dst_offset"]) + byte] ^= 1 << bit
    _, obd, otd = oracle.digest(rec, want_slab)
    ocount, omm = oracle.verify(rec, obd, want_bd, cap=64)
    fbd, ftd, count, pairs = d.fused(64)
    assert np.array_equal(fbd, obd) and np.array_equal(ftd, otd)
    assert count == ocount == 40 and pairs == [(int(m["tensor_id"]), int(m["block"])) for m in omm]
    assert d.verify(cap=64) == (count, pairs)
    d.close()


def test_geometry_is_a_multiple_of_the_sm_count():
    g = gms.gms_launch_geometry()
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    assert g["grid_ctas"] % sms == 0 and g["warps_per_cta"] >= 1 and g["smem_bytes"] <= 227 * 1024


def test_product_path_does_not_import_the_oracle():
    import paper_2609_25451_b200.gms as g

    src = open(g.__file__).read()
    assert "import oracle" not in src and "from oracle" not in src and "gms_oracle" not in src
    assert isinstance(ctypes.CDLL(g.LIB_PATH), ctypes.CDLL)
