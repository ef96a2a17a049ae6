"""GPU parity of the gather direction: gms_capture (allocations -> packed image, fused digest) and
gms_kv_capture (pool blocks -> packed image), against the CPU oracle, bit-exact, including images
in pinned mapped host memory, ragged tails, untouched gaps of the image and skipped KV ids."""
import ctypes

import numpy as np
import pytest

torch = pytest.importorskip("torch")

from paper_2609_25451_b200 import gms  # noqa: E402
from paper_2609_25451_b200 import workloads as W  # noqa: E402

from gpu_harness import CANARY, PAD, DeviceWorkload, guarded_u64, oracle_record, payload_of  # noqa: E402

FAKE_BASE = 0x7F0000000000
GAP = 0xC3  # image bytes no entry covers


def test_capture_refuses_overlapping_image_ranges_on_the_host():
    # CPU-only: restore accepts tensors that share image bytes, capture cannot
    ent = gms.make_entries([(1, 0, FAKE_BASE, 100), (2, 0, FAKE_BASE + 112, 100)])
    m = gms.gms_manifest_build(ent, 1000, gms.BUILD_HOST_ONLY)
    rc = gms.lib().gms_capture(m.handle, ctypes.c_void_p(FAKE_BASE), gms.SRC_DEVICE, None, None, None)
    assert rc == gms.ERR_OVERLAP
    ok = gms.gms_manifest_build(gms.make_entries([(1, 0, FAKE_BASE, 100), (2, 112, FAKE_BASE + 112, 100)]), 1000,
                                gms.BUILD_HOST_ONLY)
    assert gms.lib().gms_capture(ok.handle, ctypes.c_void_p(FAKE_BASE), gms.SRC_DEVICE, None, None, None) == gms.ERR_STATE
    m.close()
    ok.close()


CASES = {
    "edge": lambda: W.pack_layout("edge", [0, 1, 15, 16, 17, 4095, 4096, 4097, 8193, 65537, 131073, 3, (1 << 20) + 4097], seed=12),
    "mixed-odd": lambda: W.mixed_manifest(n_small=2000, n_large=2, large_bytes=(6 << 20) + 24, round16=False, seed=88),
    "llama8b/16": lambda: W.llama3_8b_manifest(shrink=16),
}


@pytest.mark.gpu
@pytest.mark.parametrize("name", sorted(CASES))
@pytest.mark.parametrize("host_image", [False, True])
def test_capture_parity(oracle, name, host_image):
    w = CASES[name]()
    rec = oracle_record(oracle, w)
    slab_h = W.random_bytes_host(w.slab_bytes, seed=21)
    want_img = np.full(w.image_bytes, GAP, np.uint8)
    rc, obd, otd = oracle.capture(rec, want_img, slab_h)
    assert rc == 0
    slab = torch.from_numpy(slab_h).cuda()
    d = DeviceWorkload(w, image_dev=torch.full((w.image_bytes,), GAP, dtype=torch.uint8, device="cuda"), slab=slab)
    hptr = None
    if host_image:
        hptr, target, arr = gms.gms_host_image_alloc(w.image_bytes)
        arr[:] = GAP
        kind = gms.SRC_HOST_MAPPED
    else:
        target, kind = d.image, gms.SRC_DEVICE
    try:
        d.reset_outputs()
        gms.gms_capture(d.m, target, kind, d.bd_ptr(), d.td_ptr())
        torch.cuda.synchronize()
        assert gms.gms_last_device_status(d.m) == 0
        got_img = arr.copy() if host_image else d.image.cpu().numpy()
        assert np.array_equal(got_img, want_img), "captured image (or its gaps) differ"
        assert np.array_equal(payload_of(d.bd, d.nb), obd) and np.array_equal(payload_of(d.td, d.nt), otd)
        assert np.array_equal(d.slab_host(), slab_h)  # the allocations are only read
        # restoring the captured image reproduces the allocations and the digests
        d.slab.zero_()
        bd, td = d.restore(image=target, kind=kind)
        back = d.slab_host()
        for r in w.rows:
            o, n = int(r["dst_offset"]), int(r["nbytes"])
            assert np.array_equal(back[o:o + n], slab_h[o:o + n])
        assert np.array_equal(bd, obd) and np.array_equal(td, otd)
    finally:
        torch.cuda.synchronize()
        d.close()
        if hptr:
            gms.gms_host_image_free(hptr)


def run_kv_capture(oracle, n_planes, n_blocks, block_bytes, ids, plane_gap, seed, host_image=False):
    k = block_bytes // 4096
    plane_stride = n_blocks * block_bytes + plane_gap
    n_sel = len(ids)
    ips, iss = max(n_sel, 1) * block_bytes + 64, block_bytes
    pool_h = W.random_bytes_host(n_planes * plane_stride, seed)
    want_img = np.full(n_planes * ips, GAP, np.uint8)
    rc, obd, okd, oskip = oracle.kv_capture(pool_h, plane_stride, block_bytes, n_planes, n_blocks, block_bytes, want_img, ips,
                                            iss, ids)
    assert rc == 0
    pool = torch.from_numpy(pool_h).cuda()
    hptr = None
    if host_image:
        hptr, img_ptr, arr = gms.gms_host_image_alloc(want_img.size)
        arr[:] = GAP
    else:
        img = torch.full((want_img.size,), GAP, dtype=torch.uint8, device="cuda")
        img_ptr = img.data_ptr()
    ids_d = torch.from_numpy(np.ascontiguousarray(ids, dtype=np.int32)).cuda()
    bd, kd, st = guarded_u64(n_sel * n_planes * k), guarded_u64(n_sel), guarded_u64(4)
    desc = gms.KvPool(base=pool.data_ptr(), plane_stride=plane_stride, block_stride=block_bytes, n_planes=n_planes,
                      n_blocks=n_blocks, block_bytes=block_bytes)
    gms.gms_kv_capture(desc, img_ptr, ips, iss, gms.SRC_HOST_MAPPED if host_image else gms.SRC_DEVICE, ids_d, n_sel,
                       bd.data_ptr() + 8 * PAD, kd.data_ptr() + 8 * PAD, st.data_ptr() + 8 * PAD)
    torch.cuda.synchronize()
    status = payload_of(st, 4)
    assert int(status[0]) == oskip and int(status[1]) == 0
    got = arr.copy() if host_image else img.cpu().numpy()
    assert np.array_equal(got, want_img), "captured KV image differs"
    assert np.array_equal(pool.cpu().numpy(), pool_h)  # the pool is only read
    assert np.array_equal(payload_of(bd, n_sel * n_planes * k), obd) and np.array_equal(payload_of(kd, n_sel), okd)
    assert (payload_of(kd, n_sel)[[i for i, b in enumerate(ids) if not 0 <= b < n_blocks]] == 0).all()
    if hptr:
        gms.gms_host_image_free(hptr)


@pytest.mark.gpu
def test_kv_capture_parity(oracle):
    rng = np.random.default_rng(61)
    run_kv_capture(oracle, 6, 200, 32768, rng.permutation(200)[:70].astype(np.int32), 4096, 300)
    run_kv_capture(oracle, 4, 40, 8192, np.array([5, -1, 0, 40, 39, 2**31 - 1, 7], np.int32), 0, 310)
    run_kv_capture(oracle, 3, 30, 4096, rng.permutation(30)[:12].astype(np.int32), 256, 320, host_image=True)
    assert CANARY  # canary words around every output are checked inside payload_of


@pytest.mark.gpu
def test_kv_pool_shaped_image_is_a_subset_copy_between_pools(oracle):
    """GMS_KV_IMAGE_BY_ID: the image has the pool's shape, so list position j addresses image slot ids[j].  The
    oracle knows packed images only; the packed image it is given is the pool-shaped one gathered by plain indexing."""
    rng = np.random.default_rng(91)
    n_planes, n_blocks, bb = 4, 120, 32768
    k = bb // 4096
    ids = rng.permutation(n_blocks)[:45].astype(np.int32)
    ids[5], ids[20] = -7, n_blocks  # skipped
    n_sel = len(ids)
    plane = n_blocks * bb
    a_h = W.random_bytes_host(n_planes * plane, 401)  # pool A: the "image"
    b_h = W.random_bytes_host(n_planes * plane, 402)  # pool B: the destination
    a4 = a_h.reshape(n_planes, n_blocks, bb)
    packed = np.zeros((n_planes, n_sel, bb), np.uint8)
    for j, i in enumerate(ids):
        if 0 <= i < n_blocks:
            packed[:, j] = a4[:, i]
    want_b = b_h.copy()
    rc, obd, okd, oskip = oracle.kv_restore(want_b, plane, bb, n_planes, n_blocks, bb, packed.reshape(-1), n_sel * bb, bb, ids)
    assert rc == 0 and oskip == 2
    a_d, b_d = torch.from_numpy(a_h).cuda(), torch.from_numpy(b_h).cuda()
    ids_d = torch.from_numpy(ids).cuda()
    bd, kd, st = guarded_u64(n_sel * n_planes * k), guarded_u64(n_sel), guarded_u64(4)
    desc = gms.KvPool(base=b_d.data_ptr(), plane_stride=plane, block_stride=bb, n_planes=n_planes, n_blocks=n_blocks,
                      block_bytes=bb, flags=gms.KV_IMAGE_BY_ID)
    gms.gms_kv_restore(desc, a_d, plane, bb, gms.SRC_DEVICE, ids_d, n_sel, bd.data_ptr() + 8 * PAD, kd.data_ptr() + 8 * PAD,
                       st.data_ptr() + 8 * PAD)
    torch.cuda.synchronize()
    assert payload_of(st, 4)[:2].tolist() == [2, 0]
    assert np.array_equal(b_d.cpu().numpy(), want_b) and np.array_equal(a_d.cpu().numpy(), a_h)
    assert np.array_equal(payload_of(bd, n_sel * n_planes * k), obd) and np.array_equal(payload_of(kd, n_sel), okd)
    # and back: capture B's selected blocks into a third pool-shaped buffer; only those blocks change
    c_d = torch.full((n_planes * plane,), 0x5C, dtype=torch.uint8, device="cuda")
    gms.gms_kv_capture(desc, c_d, plane, bb, gms.SRC_DEVICE, ids_d, n_sel, None, kd.data_ptr() + 8 * PAD, st.data_ptr() + 8 * PAD)
    torch.cuda.synchronize()
    want_c = np.full((n_planes, n_blocks, bb), 0x5C, np.uint8)
    for i in ids:
        if 0 <= i < n_blocks:
            want_c[:, i] = want_b.reshape(n_planes, n_blocks, bb)[:, i]
    assert np.array_equal(c_d.cpu().numpy(), want_c.reshape(-1)) and np.array_equal(payload_of(kd, n_sel), okd)
    bad = gms.KvPool(base=b_d.data_ptr(), plane_stride=plane, block_stride=bb, n_planes=n_planes, n_blocks=n_blocks,
                     block_bytes=bb, flags=0x10)
    with pytest.raises(gms.GmsError) as ei:
        gms.gms_kv_restore(bad, a_d, plane, bb, gms.SRC_DEVICE, ids_d, n_sel, None, None, st.data_ptr() + 8 * PAD)
    assert ei.value.status == gms.ERR_ARG


@pytest.mark.gpu
def test_capture_full_size_8b_round_trip(oracle):
    """At the benchmark's size: capture the 16 GB of allocations into an image, then check every image byte with
    torch, every block and tensor digest with the oracle (dealt out to one thread per host core), that digest in
    place reports the same, and that restoring the captured image gives back the allocations and the digests."""
    w = W.llama3_8b_manifest()
    slab = torch.empty(w.slab_bytes, dtype=torch.uint8, device="cuda")
    W.fill_random_device(slab, 4321)
    image = torch.zeros(w.image_bytes, dtype=torch.uint8, device="cuda")
    d = DeviceWorkload(w, image_dev=image, slab=slab)
    d.reset_outputs()
    gms.gms_capture(d.m, image, gms.SRC_DEVICE, d.bd_ptr(), d.td_ptr())
    torch.cuda.synchronize()
    bd, td = payload_of(d.bd, d.nb), payload_of(d.td, d.nt)
    for r in w.rows:
        s, o, n = int(r["src_offset"]), int(r["dst_offset"]), int(r["nbytes"])
        assert torch.equal(image[s:s + n], slab[o:o + n])
    from oracle_threads import all_digests

    rec = oracle_record(oracle, w)
    slab_h = slab.cpu().numpy()
    obd, otd = all_digests(oracle, rec, lambda t: slab_h[int(w.rows[t]["dst_offset"]):][:int(w.rows[t]["nbytes"])])
    del slab_h
    assert np.array_equal(bd, obd) and np.array_equal(td, otd)
    bd2, td2 = d.digest()
    assert np.array_equal(bd2, obd) and np.array_equal(td2, otd)
    # round trip: wipe the allocations, restore them from the captured image
    want = slab.clone()
    for r in w.rows:  # the allocations only: the bytes between them belong to nobody and restore leaves them alone
        o, n = int(r["dst_offset"]), int(r["nbytes"])
        slab[o:o + n] = 0
    bd3, td3 = d.restore()
    assert torch.equal(slab, want)
    assert np.array_equal(bd3, obd) and np.array_equal(td3, otd)
    d.close()
