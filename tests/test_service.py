"""gms_service_*: service-owned slabs with the paper's ownership protocol (EMPTY -> RW -> COMMITTED
<-> RO), a first-fit suballocator over fixed-size slabs and dedicated slabs for oversized requests.

CPU part (dry-run backend, no CUDA call): the state machine accepts exactly the transitions of the
protocol, and the allocator's addresses are aligned, disjoint, first-fit and inside their slabs.
GPU part: destinations carved from real VMM slabs take a restore (parity with the oracle), become
read-only at commit (checked through cuMemGetAccess, never by attempting a write), can still be
digested / verified / captured in place while readers hold them, and are writable again after the
last reader has left.  No test writes to a read-only mapping."""
import numpy as np
import pytest

from paper_2609_25451_b200 import gms
from paper_2609_25451_b200 import workloads as W

MiB = 1 << 20


def status_of(fn, *a):
    try:
        fn(*a)
        return gms.OK
    except gms.GmsError as e:
        return e.status


def test_ownership_state_machine_dry_run():
    s = gms.gms_service_create(8 * MiB, gms.SERVICE_DRY_RUN)
    info = lambda: gms.gms_service_info(s)
    assert info()["state"] == gms.STATE_EMPTY
    # nothing but a writer may start
    assert status_of(gms.gms_service_alloc, s, 100) == gms.ERR_STATE
    assert status_of(gms.gms_service_commit, s) == gms.ERR_STATE
    assert status_of(gms.gms_service_acquire_ro, s) == gms.ERR_STATE
    assert status_of(gms.gms_service_release_ro, s) == gms.ERR_STATE
    assert status_of(gms.gms_service_abort, s) == gms.ERR_STATE
    gms.gms_service_acquire_rw(s)
    assert info()["state"] == gms.STATE_RW
    assert status_of(gms.gms_service_acquire_rw, s) == gms.ERR_STATE  # one writer only
    assert status_of(gms.gms_service_acquire_ro, s) == gms.ERR_STATE  # no readers before commit
    p = gms.gms_service_alloc(s, 1000)
    assert gms.gms_service_access(s, p) is True
    # a writer that gives up discards everything
    gms.gms_service_abort(s)
    assert info()["state"] == gms.STATE_EMPTY and info()["n_slabs"] == 0 and info()["bytes_allocated"] == 0
    assert status_of(gms.gms_service_access, s, p) == gms.ERR_RANGE
    # populate, commit, readers come and go
    gms.gms_service_acquire_rw(s)
    p = gms.gms_service_alloc(s, 1000)
    gms.gms_service_commit(s)
    assert info()["state"] == gms.STATE_COMMITTED and gms.gms_service_access(s, p) is False
    assert status_of(gms.gms_service_alloc, s, 100) == gms.ERR_STATE  # immutable
    assert status_of(gms.gms_service_abort, s) == gms.ERR_STATE
    gms.gms_service_acquire_ro(s)
    gms.gms_service_acquire_ro(s)
    assert info()["state"] == gms.STATE_RO and info()["readers"] == 2
    assert status_of(gms.gms_service_acquire_rw, s) == gms.ERR_STATE  # readers hold it
    gms.gms_service_release_ro(s)
    assert info()["state"] == gms.STATE_RO and info()["readers"] == 1
    gms.gms_service_release_ro(s)
    assert info()["state"] == gms.STATE_COMMITTED and info()["readers"] == 0
    assert status_of(gms.gms_service_release_ro, s) == gms.ERR_STATE
    # write access returns after the last reader; contents and addresses are kept
    gms.gms_service_acquire_rw(s)
    assert info()["state"] == gms.STATE_RW and info()["n_slabs"] == 1 and gms.gms_service_access(s, p) is True
    s.close()
    assert gms.lib().gms_service_create(0, 0x80, None) == gms.ERR_NULL


def test_first_fit_suballocation_dry_run():
    slab = 8 * MiB
    s = gms.gms_service_create(slab, gms.SERVICE_DRY_RUN)
    gms.gms_service_acquire_rw(s)
    rng = np.random.default_rng(4)
    sizes = [int(x) for x in rng.integers(1, 3 * MiB, size=40)] + [slab, slab + 1, 20 * MiB, 1, 255, 256, 257]
    allocs = [(gms.gms_service_alloc(s, n), n) for n in sizes]
    info = gms.gms_service_info(s)
    assert info["slab_bytes"] == slab and info["n_dedicated"] == 2  # slab+1 and 20 MiB do not fit a regular slab
    assert info["bytes_allocated"] == sum((n + 255) // 256 * 256 for n in sizes)
    assert info["bytes_reserved"] >= info["bytes_allocated"]
    spans = sorted((p, p + (n + 255) // 256 * 256) for p, n in allocs)
    assert all(p % 256 == 0 for p, _ in spans)
    assert all(a_end <= b_start for (_, a_end), (b_start, _) in zip(spans, spans[1:]))  # pairwise disjoint
    # first fit: a small request goes into the first regular slab that still has a gap (here the very first
    # slab, whose tail was too short for the request that opened the second one), not into a new slab
    first_slab_base = allocs[0][0]
    small = gms.gms_service_alloc(s, 64)
    assert first_slab_base <= small < first_slab_base + slab
    assert gms.gms_service_info(s)["n_slabs"] == info["n_slabs"]
    assert status_of(gms.gms_service_alloc, s, 0) == gms.ERR_ARG
    s.close()


@pytest.mark.gpu
def test_restore_into_slabs_commit_read_only_and_repair(oracle):
    import torch

    from gpu_harness import oracle_record

    w = W.mixed_manifest(n_small=600, n_large=3, large_bytes=(9 * MiB) + 40, round16=False, seed=202)
    image_h = W.random_bytes_host(w.image_bytes, seed=203)
    svc = gms.gms_service_create(16 * MiB)  # small slabs so that the workload spans many of them
    gms.gms_service_acquire_rw(svc)
    ptrs = [gms.gms_service_alloc(svc, max(1, int(r["nbytes"]))) for r in w.rows]
    info = gms.gms_service_info(svc)
    assert info["n_slabs"] >= 3 and info["state"] == gms.STATE_RW
    assert all(gms.gms_service_access(svc, p) for p in ptrs[:5])
    image = torch.from_numpy(image_h).cuda()
    ent = gms.make_entries((r["tensor_id"], r["src_offset"], p, r["nbytes"]) for r, p in zip(w.rows, ptrs))
    m = gms.gms_manifest_build(ent, w.image_bytes)
    bd = torch.zeros(m.n_blocks, dtype=torch.int64, device="cuda")
    td = torch.zeros(m.n_tensors, dtype=torch.int64, device="cuda")
    gms.gms_restore(m, image, gms.SRC_DEVICE, bd, td)
    torch.cuda.synchronize()
    # the oracle's view: same record with destinations packed on the host
    rec = oracle_record(oracle, w)
    slab_h = np.zeros(w.slab_bytes, np.uint8)
    rc, obd, otd = oracle.restore(rec, image_h, slab_h)
    assert rc == 0
    assert np.array_equal(bd.cpu().numpy().view(np.uint64), obd) and np.array_equal(td.cpu().numpy().view(np.uint64), otd)
    gms.gms_manifest_set_expected(m, bd)

    # commit: every slab read-only (asked of the driver, not tried by writing)
    gms.gms_service_commit(svc)
    assert not any(gms.gms_service_access(svc, p) for p in ptrs)
    gms.gms_service_acquire_ro(svc)
    assert gms.gms_service_info(svc)["state"] == gms.STATE_RO
    # a reader digests, verifies and captures the read-only allocations in place
    bd2 = torch.zeros_like(bd)
    td2 = torch.zeros_like(td)
    gms.gms_digest(m, bd2, td2)
    out = torch.zeros(2 * 8, dtype=torch.int64, device="cuda")
    cnt = torch.full((1,), -1, dtype=torch.int64, device="cuda")
    gms.gms_verify(m, bd2, out, 8, cnt)
    back = torch.zeros(w.image_bytes, dtype=torch.uint8, device="cuda")
    gms.gms_capture(m, back, gms.SRC_DEVICE, None, None)
    torch.cuda.synchronize()
    assert torch.equal(bd2, bd) and torch.equal(td2, td) and int(cnt.item()) == 0
    for r in w.rows:
        s0, n = int(r["src_offset"]), int(r["nbytes"])
        assert torch.equal(back[s0:s0 + n], image[s0:s0 + n])
    assert gms.gms_last_device_status(m) == 0
    assert status_of(gms.gms_service_acquire_rw, svc) == gms.ERR_STATE
    gms.gms_service_release_ro(svc)

    # the last reader has left: a writer repairs in place (same addresses), with a different image
    gms.gms_service_acquire_rw(svc)
    assert all(gms.gms_service_access(svc, p) for p in ptrs)
    image2_h = W.random_bytes_host(w.image_bytes, seed=204)
    gms.gms_restore(m, torch.from_numpy(image2_h).cuda(), gms.SRC_DEVICE, bd, td)
    torch.cuda.synchronize()
    rc, obd2, otd2 = oracle.restore(rec, image2_h, slab_h)
    assert np.array_equal(bd.cpu().numpy().view(np.uint64), obd2) and np.array_equal(td.cpu().numpy().view(np.uint64), otd2)
    gms.gms_service_abort(svc)
    assert gms.gms_service_info(svc)["n_slabs"] == 0
    m.close()
    svc.close()


@pytest.mark.gpu
def test_oversized_allocation_gets_a_dedicated_slab():
    import torch

    svc = gms.gms_service_create(4 * MiB)
    gms.gms_service_acquire_rw(svc)
    small = gms.gms_service_alloc(svc, 1 * MiB)
    big = gms.gms_service_alloc(svc, 10 * MiB + 5)
    info = gms.gms_service_info(svc)
    assert info["n_slabs"] == 2 and info["n_dedicated"] == 1 and info["bytes_reserved"] >= 14 * MiB
    # both are usable device memory
    n = 10 * MiB + 5
    image = torch.from_numpy(W.random_bytes_host(n + MiB, seed=9)).cuda()
    m = gms.gms_manifest_build(gms.make_entries([(1, 0, big, n), (2, (n + 15) // 16 * 16, small, MiB - 16)]), n + MiB)
    gms.gms_restore(m, image, gms.SRC_DEVICE, None, None)
    back = torch.zeros(n + MiB, dtype=torch.uint8, device="cuda")
    gms.gms_capture(m, back, gms.SRC_DEVICE, None, None)
    torch.cuda.synchronize()
    assert torch.equal(back[:n], image[:n])
    m.close()
    svc.close()


def test_detach_and_page_release_transitions_dry_run():
    s = gms.gms_service_create(8 * MiB, gms.SERVICE_DRY_RUN)
    info = lambda: gms.gms_service_info(s)
    assert info()["attached"] == 1 and info()["backed"] == 1
    # nothing to detach or release before there is state
    for fn in (gms.gms_service_detach, gms.gms_service_reattach, gms.gms_service_release_pages, gms.gms_service_back_pages):
        assert status_of(fn, s) == gms.ERR_STATE
    gms.gms_service_acquire_rw(s)
    p = gms.gms_service_alloc(s, 5000)
    # RW: pages may be released and brought back; the books and the addresses stay
    assert status_of(gms.gms_service_detach, s) == gms.ERR_STATE
    assert status_of(gms.gms_service_back_pages, s) == gms.ERR_STATE
    gms.gms_service_release_pages(s)
    assert info()["backed"] == 0 and info()["bytes_allocated"] == 5120 and info()["n_slabs"] == 1
    assert status_of(gms.gms_service_release_pages, s) == gms.ERR_STATE
    assert status_of(gms.gms_service_alloc, s, 10) == gms.ERR_STATE
    assert status_of(gms.gms_service_commit, s) == gms.ERR_STATE
    assert status_of(gms.gms_service_access, s, p) == gms.ERR_STATE
    gms.gms_service_back_pages(s)
    assert info()["backed"] == 1 and gms.gms_service_access(s, p) is True
    q = gms.gms_service_alloc(s, 10)
    assert q != p
    gms.gms_service_commit(s)
    # COMMITTED: detach / reattach; no lease can be taken in between
    assert status_of(gms.gms_service_release_pages, s) == gms.ERR_STATE
    assert status_of(gms.gms_service_reattach, s) == gms.ERR_STATE
    gms.gms_service_detach(s)
    assert info()["attached"] == 0 and info()["state"] == gms.STATE_COMMITTED
    assert status_of(gms.gms_service_detach, s) == gms.ERR_STATE
    assert status_of(gms.gms_service_acquire_ro, s) == gms.ERR_STATE
    assert status_of(gms.gms_service_acquire_rw, s) == gms.ERR_STATE
    assert status_of(gms.gms_service_access, s, p) == gms.ERR_STATE
    gms.gms_service_reattach(s)
    assert info()["attached"] == 1 and gms.gms_service_access(s, p) is False
    gms.gms_service_acquire_ro(s)
    assert status_of(gms.gms_service_detach, s) == gms.ERR_STATE  # a reader holds it
    gms.gms_service_release_ro(s)
    # a writer that gives up while the pages are released leaves a clean, empty service
    gms.gms_service_acquire_rw(s)
    gms.gms_service_release_pages(s)
    gms.gms_service_abort(s)
    assert info()["state"] == gms.STATE_EMPTY and info()["backed"] == 1 and info()["n_slabs"] == 0
    s.close()


@pytest.mark.gpu
def test_addresses_outlive_their_mappings(oracle):
    """A manifest built once stays valid across detach / reattach (contents preserved, read-only) and across
    release_pages / back_pages (fresh memory at the same addresses, refilled by gms_restore)."""
    import torch

    from gpu_harness import oracle_record

    w = W.mixed_manifest(n_small=300, n_large=2, large_bytes=(5 * MiB) + 24, round16=False, seed=211)
    image_h = W.random_bytes_host(w.image_bytes, seed=212)
    svc = gms.gms_service_create(8 * MiB)
    gms.gms_service_acquire_rw(svc)
    ptrs = [gms.gms_service_alloc(svc, max(1, int(r["nbytes"]))) for r in w.rows]
    image = torch.from_numpy(image_h).cuda()
    m = gms.gms_manifest_build(gms.make_entries((r["tensor_id"], r["src_offset"], p, r["nbytes"]) for r, p in zip(w.rows, ptrs)),
                               w.image_bytes)
    bd = torch.zeros(m.n_blocks, dtype=torch.int64, device="cuda")
    td = torch.zeros(m.n_tensors, dtype=torch.int64, device="cuda")
    rec = oracle_record(oracle, w)
    rc, obd, otd = oracle.restore(rec, image_h, np.zeros(w.slab_bytes, np.uint8))
    assert rc == 0

    def digests_match(want_bd, want_td):
        torch.cuda.synchronize()
        assert gms.gms_last_device_status(m) == 0
        return np.array_equal(bd.cpu().numpy().view(np.uint64), want_bd) and np.array_equal(td.cpu().numpy().view(np.uint64), want_td)

    gms.gms_restore(m, image, gms.SRC_DEVICE, bd, td)
    assert digests_match(obd, otd)
    gms.gms_service_commit(svc)

    # detach: the ranges are unmapped (never touched here), the physical memory stays with the service
    gms.gms_service_detach(svc)
    assert gms.gms_service_info(svc)["attached"] == 0
    scratch = torch.empty(64 * MiB, dtype=torch.uint8, device="cuda")  # other allocations come and go meanwhile
    scratch.fill_(0xAB)
    del scratch
    gms.gms_service_reattach(svc)
    assert not any(gms.gms_service_access(svc, p) for p in ptrs)  # read-only again, same addresses
    bd.zero_()
    td.zero_()
    gms.gms_digest(m, bd, td)
    assert digests_match(obd, otd)  # contents survived

    # the memory is lost and rebuilt: fresh pages behind the same addresses, refilled from another image
    gms.gms_service_acquire_rw(svc)
    gms.gms_service_release_pages(svc)
    assert gms.gms_service_info(svc)["backed"] == 0
    gms.gms_service_back_pages(svc)
    assert all(gms.gms_service_access(svc, p) for p in ptrs)
    image2_h = W.random_bytes_host(w.image_bytes, seed=213)
    rc, obd2, otd2 = oracle.restore(rec, image2_h, np.zeros(w.slab_bytes, np.uint8))
    gms.gms_restore(m, torch.from_numpy(image2_h).cuda(), gms.SRC_DEVICE, bd, td)
    assert digests_match(obd2, otd2)
    bd.zero_()
    td.zero_()
    gms.gms_digest(m, bd, td)
    assert digests_match(obd2, otd2)
    gms.gms_service_commit(svc)
    m.close()
    svc.close()


@pytest.mark.gpu
def test_kv_pool_owned_by_the_service_is_reattached_and_checked(oracle):
    """Section 6, "Preserving KV state": for device-preserving failures the service could own the physical KV pages, so that
    KV contents stay resident and are reattached after recovery.  Here a paged KV pool lives in a slab of its own: filled in
    state RW (gms_kv_restore), committed, unmapped and mapped again at the same address (detach / reattach), then checked
    where it lies on the read-only mapping (gms_kv_digest + gms_kv_verify) -- intact; after a writer changed two blocks, the
    check names them as the oracle does.  Nothing writes through a read-only mapping."""
    import torch

    n_planes, n_blocks, bb = 6, 96, 32768
    k = bb // 4096
    plane_stride = n_blocks * bb
    pool_bytes = n_planes * plane_stride  # 18 MiB: larger than the slab size, so the pool gets a dedicated slab
    svc = gms.gms_service_create(8 * MiB)
    gms.gms_service_acquire_rw(svc)
    base = gms.gms_service_alloc(svc, pool_bytes)
    assert gms.gms_service_info(svc)["n_dedicated"] == 1
    desc = gms.KvPool(base=base, plane_stride=plane_stride, block_stride=bb, n_planes=n_planes, n_blocks=n_blocks, block_bytes=bb)
    rng = np.random.default_rng(91)
    everything = rng.permutation(n_blocks).astype(np.int32)
    image_h = W.random_bytes_host(n_planes * n_blocks * bb, seed=92)
    pool_h = np.zeros(pool_bytes, np.uint8)
    rc, _, _, _ = oracle.kv_restore(pool_h, plane_stride, bb, n_planes, n_blocks, bb, image_h, n_blocks * bb, bb, everything)
    assert rc == 0
    st = torch.zeros(4, dtype=torch.int64, device="cuda")
    gms.gms_kv_restore(desc, torch.from_numpy(image_h).cuda(), n_blocks * bb, bb, gms.SRC_DEVICE, torch.from_numpy(everything).cuda(),
                       n_blocks, None, None, st)
    torch.cuda.synchronize()
    assert st[:2].tolist() == [0, 0]

    # the committed blocks an engine would come back to: a third of the pool, in list order
    ids = rng.permutation(n_blocks)[:32].astype(np.int32)
    ids_d = torch.from_numpy(ids).cuda()
    n_slots = len(ids) * n_planes * k
    recorded = torch.zeros(n_slots, dtype=torch.int64, device="cuda")
    gms.gms_kv_digest(desc, ids_d, len(ids), recorded, None, st)
    torch.cuda.synchronize()
    rc, obd, okd, _ = oracle.kv_digest(pool_h, plane_stride, bb, n_planes, n_blocks, bb, ids)
    assert rc == 0 and np.array_equal(recorded.cpu().numpy().view(np.uint64), obd)

    def check():
        """Digest the selected blocks where they lie and compare with the recorded digests."""
        now = torch.zeros(n_slots, dtype=torch.int64, device="cuda")
        kd = torch.zeros(len(ids), dtype=torch.int64, device="cuda")
        out = torch.zeros(2 * 8, dtype=torch.int64, device="cuda")
        cnt = torch.full((1,), -1, dtype=torch.int64, device="cuda")
        scratch = torch.zeros(gms.kv_verify_scratch_words(n_slots), dtype=torch.int32, device="cuda")
        gms.gms_kv_digest(desc, ids_d, len(ids), now, kd, st)
        gms.gms_kv_verify(desc, ids_d, len(ids), now, recorded, out, 8, cnt, scratch)
        torch.cuda.synchronize()
        count = int(cnt.item())
        recs = out.cpu().numpy().view(np.uint64)[: 2 * min(count, 8)].view(gms.KV_MISMATCH_DTYPE)
        return now.cpu().numpy().view(np.uint64), kd.cpu().numpy().view(np.uint64), count, \
            [(int(r["block_id"]), int(r["plane"]), int(r["sub_block"]), int(r["list_pos"])) for r in recs]

    gms.gms_service_commit(svc)
    assert gms.gms_service_access(svc, base) is False
    gms.gms_service_detach(svc)    # the engine is gone: nothing is mapped, the pages stay with the service
    gms.gms_service_reattach(svc)  # the replacement maps them again, read-only, at the same address
    gms.gms_service_acquire_ro(svc)
    assert gms.gms_service_access(svc, base) is False
    now, kd, count, recs = check()
    assert np.array_equal(now, obd) and np.array_equal(kd, okd) and (count, recs) == (0, [])
    gms.gms_service_release_ro(svc)

    # a writer replaces two of the selected blocks (and one that is not selected); the next reader is told which
    gms.gms_service_acquire_rw(svc)
    unselected = [b for b in range(n_blocks) if b not in set(ids.tolist())]
    changed = np.array([ids[5], ids[20], unselected[0]], np.int32)
    patch_h = W.random_bytes_host(n_planes * len(changed) * bb, seed=93)
    rc, _, _, _ = oracle.kv_restore(pool_h, plane_stride, bb, n_planes, n_blocks, bb, patch_h, len(changed) * bb, bb, changed)
    assert rc == 0
    gms.gms_kv_restore(desc, torch.from_numpy(patch_h).cuda(), len(changed) * bb, bb, gms.SRC_DEVICE, torch.from_numpy(changed).cuda(),
                       len(changed), None, None, st)
    gms.gms_service_commit(svc)
    gms.gms_service_acquire_ro(svc)
    now, kd, count, recs = check()
    rc, dbd, dkd, _ = oracle.kv_digest(pool_h, plane_stride, bb, n_planes, n_blocks, bb, ids)
    ocount, orecs = oracle.kv_verify(n_planes, n_blocks, bb, ids, dbd, obd, 8)
    assert rc == 0 and np.array_equal(now, dbd) and np.array_equal(kd, dkd)
    assert ocount == 2 * n_planes * k and count == ocount  # every 4 KiB of both blocks, in every plane
    assert recs == [(int(r["block_id"]), int(r["plane"]), int(r["sub_block"]), int(r["list_pos"])) for r in orecs]
    assert {r[0] for r in recs} == {int(ids[5])}  # the first eight records all lie in the block that comes first in the list
    gms.gms_service_release_ro(svc)
    svc.close()
