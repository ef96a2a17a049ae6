"""Randomised parity soak (run by hand on a GPU machine; not collected by pytest):

    python tests/fuzz_parity.py --seconds 300 [--seed 1]

Draws random manifests (counts, size mixes, alignments, chunk lengths), random operations
(restore from device / mapped host / staged host image, digest, capture, verify after random
host-made corruption -- as separate calls and as the fused gms_digest_verify / gms_restore_verify --,
KV restore / capture / digest / verify with random ids) and compares every output with the
CPU oracle, bit for bit.  Prints one line per 50 iterations and exits non-zero on the first
difference."""
import argparse
import os
import sys
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

from oracle import gms_oracle as oracle  # noqa: E402
from paper_2609_25451_b200 import gms  # noqa: E402
from paper_2609_25451_b200 import workloads as W  # noqa: E402

from gpu_harness import CANARY, FILL, DeviceWorkload, guarded_u64, oracle_record, payload_of, PAD  # noqa: E402


def random_sizes(rng):
    kind = rng.integers(0, 5)
    n = int(rng.integers(1, 400))
    if kind == 0:  # many tiny, odd
        return [int(x) for x in rng.integers(0, 300, n)]
    if kind == 1:  # around block boundaries
        return [int(4096 * rng.integers(0, 6) + rng.integers(-17, 18)) % 30000 for _ in range(n)]
    if kind == 2:  # a few large with ragged tails
        return [int(rng.integers(1 << 18, 6 << 20)) for _ in range(int(rng.integers(1, 6)))]
    if kind == 3:  # log-uniform mix
        return [int(np.exp(rng.uniform(0, np.log(2 << 20)))) for _ in range(n)]
    return [int(rng.integers(0, 70000)) for _ in range(n)] + [int(rng.integers(1 << 20, 3 << 20))]


def one_manifest_round(rng, it):
    sizes = random_sizes(rng)
    os.environ["GMS_TUNING_HOOKS"] = "1"  # the hooks below are ignored without it
    os.environ["GMS_CHECK_TABLES"] = "1"  # device-written work lists are compared with the host's construction
    os.environ["GMS_CHUNK_BLOCKS"] = str(int(rng.choice([1, 2, 3, 4, 4, 4, 7, 16, 32])))
    os.environ["GMS_CHUNK_BLOCKS_DIGEST"] = str(int(rng.choice([1, 3, 8, 8, 8, 5, 16, 32])))
    w = W.pack_layout(f"fuzz{it}", sizes, seed=int(rng.integers(1 << 30)), guard=int(rng.choice([16, 64, 256])))
    image = W.random_bytes_host(w.image_bytes, seed=int(rng.integers(1 << 30)))
    rec = oracle_record(oracle, w)
    slab_h = np.full(w.slab_bytes, FILL, np.uint8)
    rc, obd, otd = oracle.restore(rec, image, slab_h)
    assert rc == 0
    d = DeviceWorkload(w, image)
    mode = int(rng.integers(0, 3))
    hptr = None
    if mode == 0:
        bd, td = d.restore()
    else:
        hptr, dview, arr = gms.gms_host_image_alloc(w.image_bytes)
        arr[:] = image
        if mode == 1:
            bd, td = d.restore(image=dview, kind=gms.SRC_HOST_MAPPED)
        else:
            stage = gms.gms_stage_create(int(rng.integers(2, 5)), int(rng.choice([1, 2, 8])) << 20)
            d.reset_outputs()
            gms.gms_restore_staged(d.m, stage, hptr, d.bd_ptr(), d.td_ptr())
            torch.cuda.synchronize()
            bd, td = payload_of(d.bd, d.nb), payload_of(d.td, d.nt)
            stage.close()
    assert np.array_equal(d.slab_host(), slab_h), f"restore bytes differ (mode {mode})"
    assert np.array_equal(bd, obd) and np.array_equal(td, otd), f"restore digests differ (mode {mode})"
    # corruption + digest + verify
    gms.gms_manifest_set_expected(d.m, d.bd_ptr())
    live = np.nonzero(w.rows["nbytes"] > 0)[0]
    if len(live):
        for _ in range(int(rng.integers(0, 6))):
            t = int(rng.choice(live))
            byte, bit = int(rng.integers(0, int(w.rows[t]["nbytes"]))), int(rng.integers(0, 8))
            d.flip(t, byte, bit)
            slab_h[int(w.rows[t]["dst_offset"]) + byte] ^= 1 << bit
    bd2, td2 = d.digest()
    _, obd2, otd2 = oracle.digest(rec, slab_h)
    assert np.array_equal(bd2, obd2) and np.array_equal(td2, otd2), "digest differs"
    cap = int(rng.choice([0, 1, 3, 64]))
    count, pairs = d.verify(cap=cap)
    ocount, omm = oracle.verify(rec, obd2, obd, cap=cap)
    want_pairs = [(int(m["tensor_id"]), int(m["block"])) for m in omm]
    assert count == ocount and pairs == want_pairs, "verify differs"
    # the same through the fused calls: digest + verify in one pass, then restore + verify against damaged records
    fbd, ftd, fcount, fpairs = d.fused(cap)
    assert np.array_equal(fbd, obd2) and np.array_equal(ftd, otd2) and (fcount, fpairs) == (ocount, want_pairs), "digest_verify differs"
    if rng.integers(0, 2):
        gms.gms_manifest_set_expected(d.m, d.bd_ptr())  # records of the damaged state
        fbd, ftd, fcount, fpairs = d.fused(cap, restore=True)
        ocount3, omm3 = oracle.verify(rec, obd, obd2, cap=cap)
        assert np.array_equal(fbd, obd) and np.array_equal(ftd, otd), "restore_verify digests differ"
        assert (fcount, fpairs) == (ocount3, [(int(m["tensor_id"]), int(m["block"])) for m in omm3]), "restore_verify list differs"
        slab_h2 = np.full(w.slab_bytes, FILL, np.uint8)
        oracle.restore(rec, image, slab_h2)
        assert np.array_equal(d.slab_host(), slab_h2), "restore_verify bytes differ"
        slab_h = slab_h2
        obd2, otd2 = obd, otd
    # capture the (corrupted) allocations back and compare with the oracle's capture
    want_img = np.full(w.image_bytes, 0x3C, np.uint8)
    oracle.capture(rec, want_img, slab_h)
    back = torch.full((w.image_bytes,), 0x3C, dtype=torch.uint8, device="cuda")
    d.reset_outputs()
    gms.gms_capture(d.m, back, gms.SRC_DEVICE, d.bd_ptr(), d.td_ptr())
    torch.cuda.synchronize()
    assert np.array_equal(back.cpu().numpy(), want_img), "capture bytes differ"
    assert np.array_equal(payload_of(d.bd, d.nb), obd2), "capture digests differ"
    assert gms.gms_last_device_status(d.m) == 0
    d.close()
    if hptr:
        gms.gms_host_image_free(hptr)


def one_kv_round(rng):
    n_planes, n_blocks = int(rng.integers(1, 9)), int(rng.integers(1, 200))
    bb = 4096 * int(rng.choice([1, 2, 8, 8, 32]))
    k = bb // 4096
    n_sel = int(rng.integers(0, n_blocks + 1))
    ids = rng.permutation(n_blocks)[:n_sel].astype(np.int32)
    for _ in range(int(rng.integers(0, 3))):
        if n_sel:
            ids[int(rng.integers(0, n_sel))] = int(rng.choice([-1, n_blocks, 2**31 - 1, -(2**31)]))
    gap = 16 * int(rng.integers(0, 40))
    plane_stride = n_blocks * bb + gap
    ips = max(n_sel, 1) * bb + 16 * int(rng.integers(0, 8))
    pool_h = W.random_bytes_host(n_planes * plane_stride, int(rng.integers(1 << 30)))
    img_h = W.random_bytes_host(n_planes * ips, int(rng.integers(1 << 30)))
    capture = bool(rng.integers(0, 2))
    want_pool, want_img = pool_h.copy(), img_h.copy()
    if capture:
        rc, obd, okd, oskip = oracle.kv_capture(want_pool, plane_stride, bb, n_planes, n_blocks, bb, want_img, ips, bb, ids)
    else:
        rc, obd, okd, oskip = oracle.kv_restore(want_pool, plane_stride, bb, n_planes, n_blocks, bb, want_img, ips, bb, ids)
    assert rc == 0
    pool, img = torch.from_numpy(pool_h).cuda(), torch.from_numpy(img_h).cuda()
    ids_d = torch.from_numpy(ids).cuda()
    bd, kd, st = guarded_u64(n_sel * n_planes * k), guarded_u64(n_sel), guarded_u64(4)
    desc = gms.KvPool(base=pool.data_ptr(), plane_stride=plane_stride, block_stride=bb, n_planes=n_planes, n_blocks=n_blocks,
                      block_bytes=bb)
    fn = gms.gms_kv_capture if capture else gms.gms_kv_restore
    fn(desc, img, ips, bb, gms.SRC_DEVICE, ids_d, n_sel, bd.data_ptr() + 8 * PAD, kd.data_ptr() + 8 * PAD, st.data_ptr() + 8 * PAD)
    torch.cuda.synchronize()
    status = payload_of(st, 4)
    assert int(status[0]) == oskip and int(status[1]) == 0, "kv status differs"
    assert np.array_equal(pool.cpu().numpy(), want_pool) and np.array_equal(img.cpu().numpy(), want_img), "kv bytes differ"
    assert np.array_equal(payload_of(bd, n_sel * n_planes * k), obd) and np.array_equal(payload_of(kd, n_sel), okd), "kv digests"
    # the selected blocks digested where they now lie, against the oracle's in-place digest of the expected pool
    rc, obd2, okd2, oskip2 = oracle.kv_digest(want_pool, plane_stride, bb, n_planes, n_blocks, bb, ids)
    assert rc == 0
    bd.fill_(CANARY)
    kd.fill_(CANARY)
    gms.gms_kv_digest(desc, ids_d, n_sel, bd.data_ptr() + 8 * PAD, kd.data_ptr() + 8 * PAD, st.data_ptr() + 8 * PAD)
    torch.cuda.synchronize()
    status = payload_of(st, 4)
    assert int(status[0]) == oskip2 and int(status[1]) == 0, "kv digest status differs"
    assert np.array_equal(pool.cpu().numpy(), want_pool), "kv digest wrote to the pool"
    assert np.array_equal(payload_of(bd, n_sel * n_planes * k), obd2) and np.array_equal(payload_of(kd, n_sel), okd2), "kv in-place digests"
    # host-made damage in the pool, digest again, and gms_kv_verify against the oracle's kv_verify
    n_slots = n_sel * n_planes * k
    expected = payload_of(bd, n_slots)
    exp_d = torch.from_numpy(expected.view(np.int64).copy()).cuda()
    pool_h2 = pool.cpu().numpy()
    for _ in range(int(rng.integers(0, 5))):
        pool_h2[int(rng.integers(0, pool_h2.size))] ^= 1 << int(rng.integers(0, 8))
    pool.copy_(torch.from_numpy(pool_h2))
    gms.gms_kv_digest(desc, ids_d, n_sel, bd.data_ptr() + 8 * PAD, kd.data_ptr() + 8 * PAD, st.data_ptr() + 8 * PAD)
    torch.cuda.synchronize()
    computed = payload_of(bd, n_slots)
    rc, obd3, _, _ = oracle.kv_digest(pool_h2, plane_stride, bb, n_planes, n_blocks, bb, ids)
    assert rc == 0 and np.array_equal(computed, obd3), "kv digests of the damaged pool"
    cap = int(rng.choice([0, 1, 4, 64]))
    out = torch.full((2 * cap + 2 * PAD,), CANARY, dtype=torch.int64, device="cuda")
    cnt = guarded_u64(1)
    scratch = torch.zeros(gms.kv_verify_scratch_words(n_slots), dtype=torch.int32, device="cuda")
    gms.gms_kv_verify(desc, ids_d, n_sel, bd.data_ptr() + 8 * PAD, exp_d, out.data_ptr() + 8 * PAD, cap, cnt.data_ptr() + 8 * PAD, scratch)
    torch.cuda.synchronize()
    ocount, orecs = oracle.kv_verify(n_planes, n_blocks, bb, ids, computed, expected, cap)
    count = int(payload_of(cnt, 1)[0])
    words = payload_of(out, 2 * cap)
    kk = min(count, cap)
    assert count == ocount and (words[2 * kk:] == CANARY).all(), "kv verify count"
    got = words[: 2 * kk].view(gms.KV_MISMATCH_DTYPE)
    f = ("block_id", "plane", "sub_block", "list_pos")
    assert [tuple(int(r[x]) for x in f) for r in got] == [tuple(int(r[x]) for x in f) for r in orecs], "kv verify records"


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--seconds", type=float, default=60)
    ap.add_argument("--seed", type=int, default=1)
    a = ap.parse_args()
    rng = np.random.default_rng(a.seed)
    t0, it = time.time(), 0
    while time.time() - t0 < a.seconds:
        if it % 4 == 3:
            one_kv_round(rng)
        else:
            one_manifest_round(rng, it)
        it += 1
        if it % 50 == 0:
            print(f"{it} rounds ok, {time.time() - t0:.0f} s", flush=True)
    print(f"FUZZ OK: {it} rounds in {time.time() - t0:.0f} s (seed {a.seed})")


if __name__ == "__main__":
    main()
