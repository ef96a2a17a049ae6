"""Helper run as a subprocess by test_gpu_shapes.py: the launch shape of the streaming kernels is
fixed once per process (environment hooks), so every shape needs a process of its own.  Checks
restore / digest / capture / digest + verify in one pass / kv-restore / kv-digest against the oracle on one small odd-sized workload and
prints OK."""
import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

from oracle import gms_oracle as oracle  # noqa: E402
from paper_2609_25451_b200 import gms  # noqa: E402
from paper_2609_25451_b200 import workloads as W  # noqa: E402

from gpu_harness import FILL, DeviceWorkload, oracle_record, payload_of  # noqa: E402


def main():
    w = W.mixed_manifest(n_small=1200, n_large=2, large_bytes=(5 << 20) + 24, round16=False, seed=1234)
    image = W.random_bytes_host(w.image_bytes, seed=5)
    rec = oracle_record(oracle, w)
    slab_h = np.full(w.slab_bytes, FILL, np.uint8)
    rc, obd, otd = oracle.restore(rec, image, slab_h)
    assert rc == 0
    d = DeviceWorkload(w, image)
    bd, td = d.restore()
    assert np.array_equal(d.slab_host(), slab_h) and np.array_equal(bd, obd) and np.array_equal(td, otd)
    bd, td = d.digest()
    assert np.array_equal(bd, obd) and np.array_equal(td, otd)
    back = torch.full((w.image_bytes,), 0x11, dtype=torch.uint8, device="cuda")
    d.reset_outputs()
    gms.gms_capture(d.m, back, gms.SRC_DEVICE, d.bd_ptr(), d.td_ptr())
    torch.cuda.synchronize()
    want = np.full(w.image_bytes, 0x11, np.uint8)
    oracle.capture(rec, want, slab_h)
    assert np.array_equal(back.cpu().numpy(), want) and np.array_equal(payload_of(d.bd, d.nb), obd)
    # digest + verify in one pass after host-made damage: digests, count and ordered pairs as the oracle has them
    gms.gms_manifest_set_expected(d.m, torch.from_numpy(obd.view(np.int64)).cuda())
    for row, byte, bit in W.flip_positions(w, 5, seed=21):
        d.flip(row, byte, bit)
    rc, dbd, dtd = oracle.digest(rec, d.slab_host())
    ocount, omm = oracle.verify(rec, dbd, obd, 3)
    bd, td, count, pairs = d.fused(3)
    assert np.array_equal(bd, dbd) and np.array_equal(td, dtd) and count == ocount
    assert pairs == [(int(r["tensor_id"]), int(r["block"])) for r in omm]
    d.close()
    # kv
    n_planes, n_blocks, bb = 5, 90, 32768
    ids = np.random.default_rng(3).permutation(n_blocks)[:40].astype(np.int32)
    ids[7] = -3
    pool_h = W.random_bytes_host(n_planes * n_blocks * bb, 8)
    img_h = W.random_bytes_host(n_planes * len(ids) * bb, 9)
    want_pool = pool_h.copy()
    rc, okb, okd, oskip = oracle.kv_restore(want_pool, n_blocks * bb, bb, n_planes, n_blocks, bb, img_h, len(ids) * bb, bb, ids)
    pool, img = torch.from_numpy(pool_h).cuda(), torch.from_numpy(img_h).cuda()
    kb = torch.zeros(okb.size, dtype=torch.int64, device="cuda")
    kd = torch.zeros(okd.size, dtype=torch.int64, device="cuda")
    st = torch.zeros(4, dtype=torch.int64, device="cuda")
    desc = gms.KvPool(base=pool.data_ptr(), plane_stride=n_blocks * bb, block_stride=bb, n_planes=n_planes, n_blocks=n_blocks,
                      block_bytes=bb)
    gms.gms_kv_restore(desc, img, len(ids) * bb, bb, gms.SRC_DEVICE, torch.from_numpy(ids).cuda(), len(ids), kb, kd, st)
    torch.cuda.synchronize()
    assert st[:2].tolist() == [oskip, 0] and np.array_equal(pool.cpu().numpy(), want_pool)
    assert np.array_equal(kb.cpu().numpy().view(np.uint64), okb) and np.array_equal(kd.cpu().numpy().view(np.uint64), okd)
    # the same blocks digested where they lie
    rc, dkb, dkd, dskip = oracle.kv_digest(want_pool, n_blocks * bb, bb, n_planes, n_blocks, bb, ids)
    kb.fill_(-1), kd.fill_(-1)
    gms.gms_kv_digest(desc, torch.from_numpy(ids).cuda(), len(ids), kb, kd, st)
    torch.cuda.synchronize()
    assert st[:2].tolist() == [dskip, 0] and np.array_equal(pool.cpu().numpy(), want_pool)
    assert np.array_equal(kb.cpu().numpy().view(np.uint64), dkb) and np.array_equal(kd.cpu().numpy().view(np.uint64), dkd)
    print("OK", gms.gms_launch_geometry())


if __name__ == "__main__":
    main()
