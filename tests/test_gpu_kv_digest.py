"""gms_kv_digest against the oracle: selected KV blocks digested where they lie in the pool -- the check
that decides whether KV state that outlived an engine may be reused.  Bit-exact: block digests,
per-KV-block digests, the skipped-id count; the pool must come back untouched."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

from paper_2609_25451_b200 import gms  # noqa: E402
from paper_2609_25451_b200 import workloads as W  # noqa: E402

from gpu_harness import CANARY, PAD, guarded_u64, payload_of  # noqa: E402


def run_kv_digest(oracle, n_planes, n_blocks, block_bytes, ids, plane_gap, seed, want_bd=True, want_kd=True):
    k = block_bytes // 4096
    plane_stride = n_blocks * block_bytes + plane_gap
    n_sel = len(ids)
    pool_h = W.random_bytes_host(n_planes * plane_stride, seed)
    rc, obd, okd, oskip = oracle.kv_digest(pool_h, plane_stride, block_bytes, n_planes, n_blocks, block_bytes, ids)
    assert rc == 0
    pool = torch.from_numpy(pool_h).cuda()
    ids_d = torch.from_numpy(np.ascontiguousarray(ids, dtype=np.int32)).cuda()
    bd, kd, st = guarded_u64(n_sel * n_planes * k), guarded_u64(n_sel), guarded_u64(4)
    desc = gms.KvPool(base=pool.data_ptr(), plane_stride=plane_stride, block_stride=block_bytes, n_planes=n_planes,
                      n_blocks=n_blocks, block_bytes=block_bytes)
    gms.gms_kv_digest(desc, ids_d, n_sel, bd.data_ptr() + 8 * PAD if want_bd else None,
                      kd.data_ptr() + 8 * PAD if want_kd else None, st.data_ptr() + 8 * PAD)
    torch.cuda.synchronize()
    status = payload_of(st, 4)
    assert int(status[0]) == oskip and int(status[1]) == 0
    assert np.array_equal(pool.cpu().numpy(), pool_h), "the pool was written"
    got_bd, got_kd = payload_of(bd, n_sel * n_planes * k), payload_of(kd, n_sel)
    assert np.array_equal(got_bd, obd) if want_bd else (got_bd == CANARY).all()
    assert np.array_equal(got_kd, okd) if want_kd else (got_kd == CANARY).all()
    return pool, desc, ids_d, obd, okd


def test_kv_digest_parity(oracle):
    rng = np.random.default_rng(71)
    run_kv_digest(oracle, 6, 200, 32768, rng.permutation(200)[:70].astype(np.int32), 4096, 500)
    run_kv_digest(oracle, 4, 40, 8192, np.array([5, -1, 0, 40, 39, 2**31 - 1, 7], np.int32), 0, 510)
    run_kv_digest(oracle, 3, 30, 4096, rng.permutation(30)[:12].astype(np.int32), 256, 520)
    run_kv_digest(oracle, 2, 9, 131072, np.array([8, 3, 0], np.int32), 512, 530)  # largest block size: 32 digest blocks
    run_kv_digest(oracle, 5, 64, 16384, rng.permutation(64)[:20].astype(np.int32), 0, 540, want_bd=False)
    run_kv_digest(oracle, 5, 64, 16384, rng.permutation(64)[:20].astype(np.int32), 0, 550, want_kd=False)
    run_kv_digest(oracle, 4, 16, 8192, np.zeros(0, np.int32), 0, 560)  # empty selection


def test_kv_digest_equals_what_restore_reported_and_names_a_damaged_block(oracle):
    rng = np.random.default_rng(72)
    n_planes, n_blocks, bb = 8, 150, 32768
    k = bb // 4096
    ids = rng.permutation(n_blocks)[:50].astype(np.int32)
    n_sel = len(ids)
    pool = torch.from_numpy(W.random_bytes_host(n_planes * n_blocks * bb, 600)).cuda()
    image = torch.from_numpy(W.random_bytes_host(n_planes * n_sel * bb, 601)).cuda()
    ids_d = torch.from_numpy(ids).cuda()
    nb = n_sel * n_planes * k
    bd0, bd1, kd, st = guarded_u64(nb), guarded_u64(nb), guarded_u64(n_sel), guarded_u64(4)
    desc = gms.KvPool(base=pool.data_ptr(), plane_stride=n_blocks * bb, block_stride=bb, n_planes=n_planes, n_blocks=n_blocks,
                      block_bytes=bb)
    gms.gms_kv_restore(desc, image, n_sel * bb, bb, gms.SRC_DEVICE, ids_d, n_sel, bd0.data_ptr() + 8 * PAD, None,
                       st.data_ptr() + 8 * PAD)
    # host-made damage: one bit in plane 5 of the block that slot 17 went to, inside its third 4 KiB block
    pos = 5 * n_blocks * bb + int(ids[17]) * bb + 2 * 4096 + 99
    pool[pos] = int(pool[pos].item()) ^ 0x04
    gms.gms_kv_digest(desc, ids_d, n_sel, bd1.data_ptr() + 8 * PAD, kd.data_ptr() + 8 * PAD, st.data_ptr() + 8 * PAD)
    torch.cuda.synchronize()
    a, b = payload_of(bd0, nb), payload_of(bd1, nb)
    want_slot = (17 * n_planes + 5) * k + 2
    assert np.nonzero(a != b)[0].tolist() == [want_slot]
    # gms_kv_verify names it in the block manager's terms
    assert kv_verify_gpu(desc, ids_d, n_sel, bd1.data_ptr() + 8 * PAD, bd0.data_ptr() + 8 * PAD, 4, nb) == (1, [(int(ids[17]), 5, 2, 17)])
    # the allocation-free verify names it as block `want_slot` of the flat digest array
    out = torch.full((2 * 4 + 2 * PAD,), CANARY, dtype=torch.int64, device="cuda")
    cnt = guarded_u64(1)
    gms.gms_verify_flat_noalloc(bd1.data_ptr() + 8 * PAD, bd0.data_ptr() + 8 * PAD, nb, 4242, out.data_ptr() + 8 * PAD, 4,
                                cnt.data_ptr() + 8 * PAD)
    torch.cuda.synchronize()
    assert int(payload_of(cnt, 1)[0]) == 1
    assert payload_of(out, 8)[:2].tolist() == [4242, want_slot]
    # and the oracle agrees on the damaged pool
    rc, obd, okd, _ = oracle.kv_digest(pool.cpu().numpy(), n_blocks * bb, bb, n_planes, n_blocks, bb, ids)
    assert rc == 0 and np.array_equal(b, obd) and np.array_equal(payload_of(kd, n_sel), okd)


def kv_verify_gpu(desc, ids_d, n_sel, computed, expected, cap, n_slots):
    """gms_kv_verify through the C ABI -> (count, [(block_id, plane, sub_block, list_pos), ...])."""
    out = torch.full((2 * cap + 2 * PAD,), CANARY, dtype=torch.int64, device="cuda")  # 16-byte records
    cnt = guarded_u64(1)
    scratch = torch.full((gms.kv_verify_scratch_words(n_slots) + 2,), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
    gms.gms_kv_verify(desc, ids_d, n_sel, computed, expected, out.data_ptr() + 8 * PAD, cap, cnt.data_ptr() + 8 * PAD,
                      scratch.data_ptr() + 4)
    torch.cuda.synchronize()
    assert int(scratch[0].item()) == 0x5A5A5A5A and int(scratch[-1].item()) == 0x5A5A5A5A, "scratch written out of bounds"
    count = int(payload_of(cnt, 1)[0])
    k = min(count, cap)
    words = payload_of(out, 2 * cap)
    assert (words[2 * k:] == CANARY).all(), "gms_kv_verify wrote past min(count, cap)"
    recs = words[: 2 * k].view(gms.KV_MISMATCH_DTYPE)
    return count, [(int(r["block_id"]), int(r["plane"]), int(r["sub_block"]), int(r["list_pos"])) for r in recs]


def as_tuples(recs):
    return [(int(r["block_id"]), int(r["plane"]), int(r["sub_block"]), int(r["list_pos"])) for r in recs]


@pytest.mark.parametrize("n_blocks,n_sel,n_planes,bb", [(60, 25, 4, 8192), (700, 320, 8, 32768)])
def test_kv_verify_names_damaged_blocks_like_the_oracle(oracle, n_blocks, n_sel, n_planes, bb):
    """Restore an image into a pool, damage pool bytes on the host side (some in selected blocks, some not), digest in
    place, and compare gms_kv_verify with the oracle: records, order, count, cap below the count, skipped ids.
    The small case runs the one-CTA kernel (400 slots), the large one count + emit (20,480 slots, ten segments)."""
    rng = np.random.default_rng(73 + n_blocks)
    k = bb // 4096
    ids = rng.permutation(n_blocks)[:n_sel].astype(np.int32)
    ids[3], ids[n_sel - 2] = -7, n_blocks  # two ids outside the pool: skipped, never reported
    pool = torch.from_numpy(W.random_bytes_host(n_planes * n_blocks * bb, 610)).cuda()
    image = torch.from_numpy(W.random_bytes_host(n_planes * n_sel * bb, 611)).cuda()
    ids_d = torch.from_numpy(ids).cuda()
    n_slots = n_sel * n_planes * k
    bd0, bd1, st = guarded_u64(n_slots), guarded_u64(n_slots), guarded_u64(4)
    desc = gms.KvPool(base=pool.data_ptr(), plane_stride=n_blocks * bb, block_stride=bb, n_planes=n_planes, n_blocks=n_blocks,
                      block_bytes=bb)
    gms.gms_kv_restore(desc, image, n_sel * bb, bb, gms.SRC_DEVICE, ids_d, n_sel, bd0.data_ptr() + 8 * PAD, None,
                       st.data_ptr() + 8 * PAD)
    torch.cuda.synchronize()
    assert payload_of(st, 4)[:2].tolist() == [2, 0]
    # clean: nothing to report
    gms.gms_kv_digest(desc, ids_d, n_sel, bd1.data_ptr() + 8 * PAD, None, st.data_ptr() + 8 * PAD)
    assert kv_verify_gpu(desc, ids_d, n_sel, bd1.data_ptr() + 8 * PAD, bd0.data_ptr() + 8 * PAD, 8, n_slots) == (0, [])
    # host-made damage: every 5th list position, in two planes, first and last sub-block; plus blocks not in the list
    selected = set(int(i) for i in ids if 0 <= i < n_blocks)
    pool_h = pool.cpu().numpy()
    for j in range(0, n_sel, 5):
        if not 0 <= ids[j] < n_blocks:
            continue
        for p, c in ((0, 0), (n_planes - 1, k - 1)):
            pool_h[p * n_blocks * bb + int(ids[j]) * bb + c * 4096 + int(rng.integers(0, 4096))] ^= 0x08
    for blk in [b for b in range(n_blocks) if b not in selected][:3]:
        pool_h[blk * bb + 5] ^= 0xFF
    pool.copy_(torch.from_numpy(pool_h))
    gms.gms_kv_digest(desc, ids_d, n_sel, bd1.data_ptr() + 8 * PAD, None, st.data_ptr() + 8 * PAD)
    torch.cuda.synchronize()
    computed, expected = payload_of(bd1, n_slots), payload_of(bd0, n_slots)
    rc, obd, _, _ = oracle.kv_digest(pool_h, n_blocks * bb, bb, n_planes, n_blocks, bb, ids)
    assert rc == 0 and np.array_equal(computed, obd)
    for cap in (4096, 5, 0):
        ocount, orecs = oracle.kv_verify(n_planes, n_blocks, bb, ids, computed, expected, cap)
        got = kv_verify_gpu(desc, ids_d, n_sel, bd1.data_ptr() + 8 * PAD, bd0.data_ptr() + 8 * PAD, cap, n_slots)
        assert got == (ocount, as_tuples(orecs)) and ocount >= 2 * (n_sel // 5 - 1)
    # slots of skipped ids are ignored even if the arrays differ there
    noisy = torch.from_numpy(computed.view(np.int64).copy()).cuda()
    noisy[(3 * n_planes + 1) * k] ^= 1
    noisy[((n_sel - 2) * n_planes) * k + k - 1] ^= 1
    ocount, orecs = oracle.kv_verify(n_planes, n_blocks, bb, ids, noisy.cpu().numpy().view(np.uint64), expected, 4096)
    got = kv_verify_gpu(desc, ids_d, n_sel, noisy, bd0.data_ptr() + 8 * PAD, 4096, n_slots)
    assert got == (ocount, as_tuples(orecs))
    # an empty selection reports nothing
    assert kv_verify_gpu(desc, ids_d, 0, None, None, 4, 0) == (0, [])


def test_kv_digest_argument_checks():
    pool = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    ids = torch.zeros(4, dtype=torch.int32, device="cuda")
    st = torch.zeros(4, dtype=torch.int64, device="cuda")

    def call(**kw):
        d = dict(base=pool.data_ptr(), plane_stride=1 << 19, block_stride=8192, n_planes=2, n_blocks=64, block_bytes=8192)
        d.update(kw)
        try:
            gms.gms_kv_digest(gms.KvPool(**d), ids, 4, None, None, st)
        except gms.GmsError as e:
            return e.status
        return gms.OK

    assert call() == gms.OK
    assert call(block_bytes=1000) == gms.ERR_ALIGN
    assert call(block_bytes=1 << 18) == gms.ERR_ARG
    assert call(plane_stride=(1 << 19) + 8) == gms.ERR_ALIGN
    assert call(base=None) == gms.ERR_NULL
    assert call(block_stride=4096) == gms.ERR_ARG
    assert call(plane_stride=63 * 8192 + 8192 - 16) == gms.ERR_ARG  # planes would share bytes
    torch.cuda.synchronize()
