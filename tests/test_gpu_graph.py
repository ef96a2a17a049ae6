"""The entry points only enqueue work on the caller's stream, so a recovery step can be captured
into a CUDA graph once and replayed: the replays must give the oracle's bytes and digests for
whatever the image buffer holds at replay time (the graph fixes addresses, not contents)."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

from paper_2609_25451_b200 import gms  # noqa: E402
from paper_2609_25451_b200 import workloads as W  # noqa: E402

from gpu_harness import CANARY, FILL, PAD, DeviceWorkload, guarded_u64, oracle_record, payload_of  # noqa: E402


def _warm(fn):
    """Runs fn once on a side stream (first-call set-up must not happen inside a capture)."""
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        fn()
    torch.cuda.current_stream().wait_stream(s)
    torch.cuda.synchronize()


def test_restore_verify_digest_replay_from_a_graph(oracle):
    w = W.mixed_manifest(n_small=1500, n_large=2, large_bytes=(4 << 20) + 40, round16=False)
    rec = oracle_record(oracle, w)
    image_a = W.random_bytes_host(w.image_bytes, seed=71)
    image_b = image_a.copy()
    for row, byte, bit in W.flip_positions(w, 4, seed=9):  # the second image differs in four blocks
        image_b[int(w.rows[row]["src_offset"]) + byte] ^= 1 << bit

    def want(image):
        slab = np.full(w.slab_bytes, FILL, np.uint8)
        rc, bd, td = oracle.restore(rec, image, slab)
        assert rc == 0
        return slab, bd, td

    slab_a, bd_a, td_a = want(image_a)
    slab_b, bd_b, td_b = want(image_b)

    d = DeviceWorkload(w, image_a)
    expected = torch.from_numpy(bd_a.view(np.int64).copy()).cuda()
    gms.gms_manifest_set_expected(d.m, expected.data_ptr())
    cap = 16
    out = torch.full((2 * cap + 2 * PAD,), CANARY, dtype=torch.int64, device="cuda")
    cnt = guarded_u64(1)
    bd2, td2 = guarded_u64(d.nb), guarded_u64(d.nt)

    def step():
        gms.gms_restore(d.m, d.image, gms.SRC_DEVICE, d.bd_ptr(), d.td_ptr())
        gms.gms_verify(d.m, d.bd_ptr(), out.data_ptr() + 8 * PAD, cap, cnt.data_ptr() + 8 * PAD)
        gms.gms_digest(d.m, bd2.data_ptr() + 8 * PAD, td2.data_ptr() + 8 * PAD)

    _warm(step)
    launches0 = gms.gms_kernel_launches()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    per_step = gms.gms_kernel_launches() - launches0
    assert per_step >= 5  # two streaming kernels with their prologues, and the verify

    for image, slab_w, bd_w, td_w in ((image_a, slab_a, bd_a, td_a), (image_b, slab_b, bd_b, td_b), (image_a, slab_a, bd_a, td_a)):
        d.image.copy_(torch.from_numpy(image))
        d.slab.fill_(FILL)
        for t in (d.bd, d.td, bd2, td2, out, cnt):
            t.fill_(CANARY)
        graph.replay()
        torch.cuda.synchronize()
        assert gms.gms_last_device_status(d.m) == 0
        assert np.array_equal(d.slab_host(), slab_w)
        assert np.array_equal(payload_of(d.bd, d.nb), bd_w) and np.array_equal(payload_of(d.td, d.nt), td_w)
        assert np.array_equal(payload_of(bd2, d.nb), bd_w) and np.array_equal(payload_of(td2, d.nt), td_w)
        ocount, omm = oracle.verify(rec, bd_w, bd_a, cap=cap)
        assert int(payload_of(cnt, 1)[0]) == ocount
        pairs = payload_of(out, 2 * cap).reshape(cap, 2)
        assert [(int(a), int(b)) for a, b in pairs[:ocount]] == [(int(m["tensor_id"]), int(m["block"])) for m in omm]
        assert (pairs[ocount:] == CANARY).all()
    assert ocount == 0  # the last replay restored the recorded image again
    d.close()


def test_fused_calls_replay_from_a_graph(oracle):
    """gms_restore_verify + gms_digest_verify captured once (5 kernel nodes less than the separate calls need) and
    replayed over images that differ from the recorded one in a few blocks: digests, list and count from the oracle."""
    w = W.mixed_manifest(n_small=2500, n_large=4, large_bytes=(12 << 20) + 24, round16=False, seed=91)  # > 16 K blocks
    rec = oracle_record(oracle, w)
    image_a = W.random_bytes_host(w.image_bytes, seed=72)
    image_b = image_a.copy()
    for row, byte, bit in W.flip_positions(w, 5, seed=10):
        image_b[int(w.rows[row]["src_offset"]) + byte] ^= 1 << bit

    def want(image):
        slab = np.full(w.slab_bytes, FILL, np.uint8)
        rc, bd, td = oracle.restore(rec, image, slab)
        assert rc == 0
        return slab, bd, td

    slab_a, bd_a, td_a = want(image_a)
    slab_b, bd_b, td_b = want(image_b)
    d = DeviceWorkload(w, image_a)
    assert d.nb > 16384  # the emit kernel runs over several segments
    expected = torch.from_numpy(bd_a.view(np.int64).copy()).cuda()
    gms.gms_manifest_set_expected(d.m, expected.data_ptr())
    cap = 16
    out1 = torch.full((2 * cap + 2 * PAD,), CANARY, dtype=torch.int64, device="cuda")
    out2 = torch.full((2 * cap + 2 * PAD,), CANARY, dtype=torch.int64, device="cuda")
    cnt1, cnt2 = guarded_u64(1), guarded_u64(1)
    bd2, td2 = guarded_u64(d.nb), guarded_u64(d.nt)

    def step():
        gms.gms_restore_verify(d.m, d.image, gms.SRC_DEVICE, d.bd_ptr(), d.td_ptr(), out1.data_ptr() + 8 * PAD, cap,
                               cnt1.data_ptr() + 8 * PAD)
        gms.gms_digest_verify(d.m, bd2.data_ptr() + 8 * PAD, td2.data_ptr() + 8 * PAD, out2.data_ptr() + 8 * PAD, cap,
                              cnt2.data_ptr() + 8 * PAD)

    _warm(step)
    launches0 = gms.gms_kernel_launches()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    assert gms.gms_kernel_launches() - launches0 == 6  # per call: prologue, streaming kernel, emit

    for image, slab_w, bd_w, td_w in ((image_b, slab_b, bd_b, td_b), (image_a, slab_a, bd_a, td_a), (image_b, slab_b, bd_b, td_b)):
        d.image.copy_(torch.from_numpy(image))
        d.slab.fill_(FILL)
        for t in (d.bd, d.td, bd2, td2, out1, out2, cnt1, cnt2):
            t.fill_(CANARY)
        graph.replay()
        torch.cuda.synchronize()
        assert gms.gms_last_device_status(d.m) == 0
        assert np.array_equal(d.slab_host(), slab_w)
        ocount, omm = oracle.verify(rec, bd_w, bd_a, cap=cap)
        want_pairs = [(int(m["tensor_id"]), int(m["block"])) for m in omm]
        for bdt, tdt, out, cnt in ((d.bd, d.td, out1, cnt1), (bd2, td2, out2, cnt2)):
            assert np.array_equal(payload_of(bdt, d.nb), bd_w) and np.array_equal(payload_of(tdt, d.nt), td_w)
            assert int(payload_of(cnt, 1)[0]) == ocount
            pairs = payload_of(out, 2 * cap).reshape(cap, 2)
            assert [(int(a), int(b)) for a, b in pairs[:ocount]] == want_pairs and (pairs[ocount:] == CANARY).all()
    assert ocount == 5
    d.close()


def test_kv_restore_replays_from_a_graph_with_new_block_ids(oracle):
    n_planes, n_blocks, block_bytes, n_sel = 4, 96, 16384, 40
    rng = np.random.default_rng(5)
    plane_stride = n_blocks * block_bytes + 4096
    pool = torch.full((n_planes * plane_stride,), FILL, dtype=torch.uint8, device="cuda")
    image_h = W.random_bytes_host(n_planes * n_sel * block_bytes, seed=33)
    image = torch.from_numpy(image_h).cuda()
    ids = torch.zeros(n_sel, dtype=torch.int32, device="cuda")
    bpb = block_bytes // 4096
    bd = guarded_u64(n_planes * n_sel * bpb)
    kd = guarded_u64(n_sel)
    status = torch.zeros(4, dtype=torch.int64, device="cuda")
    kvp = gms.KvPool(base=pool.data_ptr(), plane_stride=plane_stride, block_stride=block_bytes, n_planes=n_planes,
                     n_blocks=n_blocks, block_bytes=block_bytes)

    def step():
        gms.gms_kv_restore(kvp, image.data_ptr(), n_sel * block_bytes, block_bytes, gms.SRC_DEVICE, ids, n_sel,
                           bd.data_ptr() + 8 * PAD, kd.data_ptr() + 8 * PAD, status)

    _warm(step)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()

    for _ in range(3):
        ids_h = rng.permutation(n_blocks)[:n_sel].astype(np.int32)
        ids_h[rng.integers(0, n_sel)] = n_blocks + 3  # one id out of range: skipped and counted
        ids.copy_(torch.from_numpy(ids_h))
        pool.fill_(FILL)
        bd.fill_(CANARY)
        kd.fill_(CANARY)
        graph.replay()
        torch.cuda.synchronize()
        pool_w = np.full(n_planes * plane_stride, FILL, np.uint8)
        rc, obd, okd, skipped = oracle.kv_restore(pool_w, plane_stride, block_bytes, n_planes, n_blocks, block_bytes, image_h,
                                                  n_sel * block_bytes, block_bytes, ids_h)
        assert rc == 0 and skipped == 1
        st = status.cpu().numpy().view(np.uint64)
        assert int(st[0]) == 1 and int(st[1]) == 0
        assert np.array_equal(pool.cpu().numpy(), pool_w)
        assert np.array_equal(payload_of(bd, obd.size), obd) and np.array_equal(payload_of(kd, n_sel), okd)
