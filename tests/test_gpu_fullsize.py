"""Parity at the benchmark's full sizes, in the launch configuration bench.py times (library
defaults).  Every digest the library reports is compared with the oracle's: the single-threaded
oracle does about 1.1 GB/s per core, so its calls are dealt out to one thread per host core
(tests/oracle_threads.py) and the 16-34 GB workloads take it a few seconds.  Each test combines
  * exact whole-output properties checked on the device with plain torch ops (every destination
    byte equals its image byte, nothing else in the slab/pool changed), with
  * the oracle's block and tensor (or KV-block) digests of the whole workload, compared as entire
    arrays,
  * host-made single-bit flips that gms_verify must name exactly.
The mixed manifest (2.3 GB) also goes through the oracle's restore itself, in both its
16-byte-rounded and raw odd-sized forms."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

from paper_2609_25451_b200 import gms  # noqa: E402
from paper_2609_25451_b200 import workloads as W  # noqa: E402

from gpu_harness import FILL, DeviceWorkload, oracle_record  # noqa: E402
from oracle_threads import all_digests, all_kv_digests  # noqa: E402


def u64(t):
    return t.cpu().numpy().view(np.uint64)


def expected_slab(w, image):
    exp = torch.full((w.slab_bytes,), FILL, dtype=torch.uint8, device="cuda")
    for r in w.rows:
        s, d, n = int(r["src_offset"]), int(r["dst_offset"]), int(r["nbytes"])
        exp[d:d + n] = image[s:s + n]
    return exp


def check_sampled_blocks(oracle, w, image, bd, base, rng, n_samples):
    live = np.nonzero(w.rows["nbytes"] > 0)[0]
    for _ in range(n_samples):
        t = int(rng.choice(live))
        n = int(w.rows[t]["nbytes"])
        b = int(rng.integers(0, (n + 4095) // 4096))
        if rng.random() < 0.2:
            b = (n + 4095) // 4096 - 1  # favour ragged last blocks
        lo, hi = b * 4096, min(n, b * 4096 + 4096)
        s = int(w.rows[t]["src_offset"])
        want = oracle.block_digest(image[s + lo:s + hi].cpu().numpy())
        assert int(bd[int(base[t]) + b]) == want, (t, b)


def test_llama3_8b_manifest_full_size(oracle):
    w = W.llama3_8b_manifest()
    image = torch.empty(w.image_bytes, dtype=torch.uint8, device="cuda")
    W.fill_random_device(image, 991)
    d = DeviceWorkload(w, image_dev=image)
    bd, td = d.restore()
    # every destination byte, every guard band
    exp = expected_slab(w, image)
    assert torch.equal(d.slab, exp)
    del exp
    # the oracle's digests of the whole image: all 3,921,026 blocks and all 291 tensors
    rec = oracle_record(oracle, w)
    base, total = oracle.block_bases(rec)
    assert total == bd.size == 3_921_026
    image_h = image.cpu().numpy()
    obd, otd = all_digests(oracle, rec, lambda t: image_h[int(w.rows[t]["src_offset"]):][:int(w.rows[t]["nbytes"])])
    del image_h
    assert np.array_equal(bd, obd) and np.array_equal(td, otd)
    # digest in place reports the same, and so do the fused calls
    bd2, td2 = d.digest()
    assert np.array_equal(bd2, obd) and np.array_equal(td2, otd)
    # verify: clean, then 3 host-made single-bit flips
    gms.gms_manifest_set_expected(d.m, d.bd_ptr())
    assert d.verify(cap=8) == (0, [])
    fbd, ftd, fcount, fpairs = d.fused(8)
    assert np.array_equal(fbd, obd) and np.array_equal(ftd, otd) and (fcount, fpairs) == (0, [])
    flips = W.flip_positions(w, 3, seed=23)
    for row, byte, bit in flips:
        d.flip(row, byte, bit)
    bd3, td3 = d.digest()
    count, pairs = d.verify(cap=8)
    want = sorted(((row, byte // 4096) for row, byte, _ in flips))
    assert count == 3 and pairs == [(int(w.rows[r]["tensor_id"]), b) for r, b in want]
    ocount, omm = oracle.verify(rec, bd3, obd, 8)  # the oracle's verdict on the same two digest arrays
    assert ocount == 3 and pairs == [(int(m["tensor_id"]), int(m["block"])) for m in omm]
    changed = np.nonzero(bd3 != bd)[0].tolist()
    assert changed == [int(base[r]) + b for r, b in want]
    assert sorted(np.nonzero(td3 != td)[0].tolist()) == sorted({r for r, _ in want})
    # the damaged blocks' digests are the oracle's digests of the damaged bytes
    for r, b in want:
        n, o = int(w.rows[r]["nbytes"]), int(w.rows[r]["dst_offset"])
        assert int(bd3[int(base[r]) + b]) == oracle.block_digest(d.slab[o + b * 4096:o + min(n, b * 4096 + 4096)].cpu().numpy())
    fbd, ftd, fcount, fpairs = d.fused(8)
    assert np.array_equal(fbd, bd3) and np.array_equal(ftd, td3) and (fcount, fpairs) == (3, pairs)
    # restore + verify in one pass repairs the damage and reports the oracle's digests again
    fbd, ftd, fcount, fpairs = d.fused(8, restore=True)
    assert np.array_equal(fbd, obd) and np.array_equal(ftd, otd) and (fcount, fpairs) == (0, [])
    d.close()


def test_llama3_8b_manifest_fed_from_a_file_and_from_a_pinned_image(oracle, tmp_path):
    """The 16 GB manifest restored twice more without a resident device image: through gms_restore_fd (file ->
    pinned ring -> kernel) and gms_restore_staged (pinned image -> copy engine -> device ring -> kernel).  Both must
    leave exactly the bytes and digests of the plain device-staged restore; sampled blocks are checked with the oracle."""
    import os
    import shutil

    w = W.llama3_8b_manifest()
    shm = "/dev/shm" if os.path.isdir("/dev/shm") and shutil.disk_usage("/dev/shm").free > w.image_bytes + (2 << 30) else None
    if shm is None and shutil.disk_usage(str(tmp_path)).free < w.image_bytes + (2 << 30):
        pytest.skip("no room for a 16 GB snapshot file")
    try:
        hptr, _, arr = gms.gms_host_image_alloc(w.image_bytes)
    except gms.GmsError as e:
        pytest.skip(f"cannot pin 16 GB of host memory here: {e}")
    path = os.path.join(shm or str(tmp_path), f"gms_test_image_{os.getpid()}.bin")
    try:
        image = torch.empty(w.image_bytes, dtype=torch.uint8, device="cuda")
        W.fill_random_device(image, 996)
        cpu = torch.from_numpy(arr)
        for a in range(0, w.image_bytes, 1 << 30):
            cpu[a:a + (1 << 30)].copy_(image[a:a + (1 << 30)])
        with open(path, "wb") as f:
            for a in range(0, w.image_bytes, 1 << 30):
                f.write(arr[a:a + (1 << 30)].tobytes())
        d = DeviceWorkload(w, image_dev=image)
        bd, td = d.restore()
        want = d.slab.clone()
        rec = oracle_record(oracle, w)
        base, _ = oracle.block_bases(rec)
        check_sampled_blocks(oracle, w, image, bd, base, np.random.default_rng(41), 100)
        del image
        d.image = torch.zeros(16, dtype=torch.uint8, device="cuda")  # no device image from here on

        pipe = gms.gms_pipe_create(4, 256 << 20, 16)
        fd = os.open(path, os.O_RDONLY)
        d.slab.fill_(FILL)
        d.reset_outputs()
        st = gms.gms_restore_fd(d.m, pipe, fd, 0, d.bd_ptr(), d.td_ptr())
        os.close(fd)
        pipe.close()
        from gpu_harness import payload_of

        assert torch.equal(d.slab, want) and st["bytes_read"] <= w.image_bytes
        assert np.array_equal(payload_of(d.bd, d.nb), bd) and np.array_equal(payload_of(d.td, d.nt), td)

        stage = gms.gms_stage_create(3, 64 << 20)
        d.slab.fill_(FILL)
        d.reset_outputs()
        gms.gms_restore_staged(d.m, stage, hptr, d.bd_ptr(), d.td_ptr())
        torch.cuda.synchronize()
        assert torch.equal(d.slab, want)
        assert np.array_equal(payload_of(d.bd, d.nb), bd) and np.array_equal(payload_of(d.td, d.nt), td)
        assert gms.gms_last_device_status(d.m) == 0
        stage.close()
        d.close()
    finally:
        torch.cuda.synchronize()
        if os.path.exists(path):
            os.remove(path)
        gms.gms_host_image_free(hptr)


def test_single_tensor_beyond_4_gib(oracle):
    """One tensor of 4 GiB + 4 KiB + 1 bytes (more than 2^20 blocks, byte offsets beyond 32 bits, ragged tail):
    every byte on the device, the whole tensor digest and sampled block digests against the oracle."""
    n = (4 << 30) + 4096 + 1
    w = W.pack_layout("huge", [48, n, 16], seed=6)
    image = torch.empty(w.image_bytes, dtype=torch.uint8, device="cuda")
    W.fill_random_device(image, 995)
    d = DeviceWorkload(w, image_dev=image)
    bd, td = d.restore()
    assert torch.equal(d.slab, expected_slab(w, image))
    bd2, td2 = d.digest()
    assert np.array_equal(bd, bd2) and np.array_equal(td, td2)
    rec = oracle_record(oracle, w)
    base, total = oracle.block_bases(rec)
    assert total == 1 + (1 << 20) + 2 + 1
    s = int(w.rows[1]["src_offset"])
    T, obd = oracle.tensor_digest(image[s:s + n].cpu().numpy())  # ~3 s of oracle time
    assert int(td[1]) == T
    assert np.array_equal(bd[int(base[1]):int(base[1]) + obd.size], obd)
    for t in (0, 2):
        s0, n0 = int(w.rows[t]["src_offset"]), int(w.rows[t]["nbytes"])
        T0, _ = oracle.tensor_digest(image[s0:s0 + n0].cpu().numpy())
        assert int(td[t]) == T0
    # a flip in the very last byte (offset 2^32 + 4096) is named with its block index 2^20 + 1
    gms.gms_manifest_set_expected(d.m, d.bd_ptr())
    d.flip(1, n - 1, 7)
    d.digest()
    assert d.verify(cap=4) == (1, [(int(w.rows[1]["tensor_id"]), (1 << 20) + 1)])
    d.close()


@pytest.mark.parametrize("round16", [True, False])
def test_mixed_manifest_full_size_against_the_oracle_in_full(oracle, round16):
    w = W.mixed_manifest(round16=round16)
    image = torch.empty(w.image_bytes, dtype=torch.uint8, device="cuda")
    W.fill_random_device(image, 992 + round16)
    image_h = image.cpu().numpy()
    slab_h = np.full(w.slab_bytes, FILL, np.uint8)
    rc, obd, otd = oracle.restore(oracle_record(oracle, w), image_h, slab_h)
    assert rc == 0
    d = DeviceWorkload(w, image_dev=image)
    bd, td = d.restore()
    assert torch.equal(d.slab, torch.from_numpy(slab_h).cuda())
    assert np.array_equal(bd, obd) and np.array_equal(td, otd)
    bd2, td2 = d.digest()
    assert np.array_equal(bd2, obd) and np.array_equal(td2, otd)
    d.close()


def test_kv_pool_full_size(oracle):
    k = W.kv_pool_workload()
    pool = torch.empty(k.pool_bytes, dtype=torch.uint8, device="cuda")
    W.fill_random_device(pool, 993)
    image = torch.empty(k.image_bytes, dtype=torch.uint8, device="cuda")
    W.fill_random_device(image, 994)
    kk = k.block_bytes // 4096
    n_sel = len(k.ids)
    # wrapping 64-bit sum of every pool block before the call (any changed bit changes the sum)
    sums_before = pool.view(torch.int64).view(k.n_planes * k.n_blocks, -1).sum(dim=1)
    ids = torch.from_numpy(k.ids).cuda()
    bd = torch.zeros(n_sel * k.n_planes * kk, dtype=torch.int64, device="cuda")
    kd = torch.zeros(n_sel, dtype=torch.int64, device="cuda")
    st = torch.full((4,), -1, dtype=torch.int64, device="cuda")
    desc = gms.KvPool(base=pool.data_ptr(), plane_stride=k.plane_stride, block_stride=k.block_stride, n_planes=k.n_planes,
                      n_blocks=k.n_blocks, block_bytes=k.block_bytes)
    gms.gms_kv_restore(desc, image, k.img_plane_stride, k.img_slot_stride, gms.SRC_DEVICE, ids, n_sel, bd, kd, st)
    torch.cuda.synchronize()
    assert st[:2].tolist() == [0, 0]
    pool3 = pool.view(k.n_planes, k.n_blocks, k.block_bytes)
    img3 = image.view(k.n_planes, n_sel, k.block_bytes)
    for p in range(k.n_planes):  # every selected block equals its image slot
        assert torch.equal(pool3[p].index_select(0, ids.long()), img3[p]), p
    sums_after = pool.view(torch.int64).view(k.n_planes * k.n_blocks, -1).sum(dim=1)
    untouched = torch.ones(k.n_planes, k.n_blocks, dtype=torch.bool, device="cuda")
    untouched[:, ids.long()] = False
    assert torch.equal(sums_after.view(k.n_planes, k.n_blocks)[untouched], sums_before.view(k.n_planes, k.n_blocks)[untouched])
    # the oracle on every slot: all 1,464,832 block digests and all 2,861 KV-block digests
    img_h = image.cpu().numpy().reshape(k.n_planes, n_sel, k.block_bytes)
    obd, okd = all_kv_digests(oracle, n_sel, k.n_planes, k.block_bytes, lambda j: np.ascontiguousarray(img_h[:, j, :]).reshape(-1))
    del img_h
    assert obd.size == 1_464_832
    assert np.array_equal(u64(bd), obd) and np.array_equal(u64(kd), okd)
    # digesting the same blocks where they now lie gives the same digests and writes nothing
    bd2, kd2 = torch.zeros_like(bd), torch.zeros_like(kd)
    gms.gms_kv_digest(desc, ids, n_sel, bd2, kd2, st)
    torch.cuda.synchronize()
    assert st[:2].tolist() == [0, 0]
    assert np.array_equal(u64(bd2), obd) and np.array_equal(u64(kd2), okd)
    assert torch.equal(pool.view(torch.int64).view(k.n_planes * k.n_blocks, -1).sum(dim=1), sums_after)
    # nothing to report; then one host-made flip, named by block id, plane and sub-block as the oracle names it
    out = torch.zeros(2 * 8, dtype=torch.int64, device="cuda")
    cnt = torch.full((1,), -1, dtype=torch.int64, device="cuda")
    scratch = torch.zeros(gms.kv_verify_scratch_words(obd.size), dtype=torch.int32, device="cuda")
    gms.gms_kv_verify(desc, ids, n_sel, bd2, bd, out, 8, cnt, scratch)
    torch.cuda.synchronize()
    assert int(cnt.item()) == 0
    j, p, c = 1234, 41, 5
    pos = p * k.plane_stride + int(k.ids[j]) * k.block_stride + c * 4096 + 77
    pool[pos] = int(pool[pos].item()) ^ 0x02
    gms.gms_kv_digest(desc, ids, n_sel, bd2, kd2, st)
    gms.gms_kv_verify(desc, ids, n_sel, bd2, bd, out, 8, cnt, scratch)
    torch.cuda.synchronize()
    ocount, orecs = oracle.kv_verify(k.n_planes, k.n_blocks, k.block_bytes, k.ids, u64(bd2), obd, 8)
    assert int(cnt.item()) == ocount == 1
    got = out[:2].cpu().numpy().view(gms.KV_MISMATCH_DTYPE)[0]
    assert tuple(int(got[f]) for f in ("block_id", "plane", "sub_block", "list_pos")) == (int(k.ids[j]), p, c, j)
    assert tuple(int(orecs[0][f]) for f in ("block_id", "plane", "sub_block", "list_pos")) == (int(k.ids[j]), p, c, j)


def test_host_sourced_70b_shard_full_size(oracle):
    w = W.llama3_70b_tp8_shard_manifest(image_bytes=32 << 30)
    try:
        hptr, dview, arr = gms.gms_host_image_alloc(w.image_bytes)
    except gms.GmsError as e:  # the box may not allow 32 GiB of pinned memory
        pytest.skip(f"cannot pin 32 GiB of host memory here: {e}")
    try:
        cpu = torch.from_numpy(arr)
        scratch = torch.empty(1 << 30, dtype=torch.uint8, device="cuda")
        for i, a in enumerate(range(0, w.image_bytes, 1 << 30)):
            n = min(1 << 30, w.image_bytes - a)
            W.fill_random_device(scratch[:n], 7000 + i)
            cpu[a:a + n].copy_(scratch[:n])
        del scratch
        slab = torch.full((w.slab_bytes,), FILL, dtype=torch.uint8, device="cuda")
        d = DeviceWorkload(w, image_dev=torch.zeros(16, dtype=torch.uint8, device="cuda"), slab=slab)
        bd, td = d.restore(image=dview, kind=gms.SRC_HOST_MAPPED)
        # every destination byte against the host image (uploaded tensor by tensor), guards included
        covered = torch.zeros(w.slab_bytes, dtype=torch.bool, device="cuda")
        for r in w.rows:
            s, dd, n = int(r["src_offset"]), int(r["dst_offset"]), int(r["nbytes"])
            assert torch.equal(slab[dd:dd + n], cpu[s:s + n].cuda()), int(r["tensor_id"])
            covered[dd:dd + n] = True
        assert bool((slab[~covered] == FILL).all())
        del covered
        # the oracle's digests of the whole 34.3 GB host image: every block and every one of the 1,413 tensors
        rec = oracle_record(oracle, w)
        obd, otd = all_digests(oracle, rec, lambda t: arr[int(w.rows[t]["src_offset"]):][:int(w.rows[t]["nbytes"])])
        assert np.array_equal(bd, obd) and np.array_equal(td, otd)
        bd2, td2 = d.digest()
        assert np.array_equal(bd2, obd) and np.array_equal(td2, otd)
        # the copy-engine-fed restore of the same image reports the same
        stage = gms.gms_stage_create(3, 64 << 20)
        slab.fill_(FILL)
        d.reset_outputs()
        gms.gms_restore_staged(d.m, stage, hptr, d.bd_ptr(), d.td_ptr())
        torch.cuda.synchronize()
        from gpu_harness import payload_of

        assert np.array_equal(payload_of(d.bd, d.nb), obd) and np.array_equal(payload_of(d.td, d.nt), otd)
        assert gms.gms_last_device_status(d.m) == 0
        bd3, td3 = d.digest()  # the bytes it left are the bytes the oracle digested
        assert np.array_equal(bd3, obd) and np.array_equal(td3, otd)
        stage.close()
        d.close()
    finally:
        torch.cuda.synchronize()
        gms.gms_host_image_free(hptr)
