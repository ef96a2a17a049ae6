"""The calls strung together the way a recovery uses them (Sections 2.2, 3.2, 3.3): a writer populates
service-owned allocations from a snapshot image and commits them with their digests; after an engine
loss a replacement attaches read-only, digests the surviving allocations in place and decides from
gms_verify whether they can be reused; damaged tensors (damage made by the host while a writer holds
the service -- nothing here writes through a read-only mapping) are named exactly, and a writer
repairs only those from the image through a manifest of the damaged entries.  Every digest and every
repaired byte is checked against the CPU oracle."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

from paper_2609_25451_b200 import gms  # noqa: E402
from paper_2609_25451_b200 import workloads as W  # noqa: E402

from gpu_harness import oracle_record  # noqa: E402

MiB = 1 << 20


def test_commit_reuse_detect_and_partial_repair(oracle):
    w = W.mixed_manifest(n_small=500, n_large=3, large_bytes=(6 * MiB) + 8, round16=False, seed=301)
    image_h = W.random_bytes_host(w.image_bytes, seed=302)
    image = torch.from_numpy(image_h).cuda()
    rec = oracle_record(oracle, w)
    rc, obd, otd = oracle.restore(rec, image_h, np.zeros(w.slab_bytes, np.uint8))
    assert rc == 0

    # ---- cold start: the writer populates and commits
    svc = gms.gms_service_create(8 * MiB)
    gms.gms_service_acquire_rw(svc)
    ptrs = [gms.gms_service_alloc(svc, max(1, int(r["nbytes"]))) for r in w.rows]
    entries = gms.make_entries((r["tensor_id"], r["src_offset"], p, r["nbytes"]) for r, p in zip(w.rows, ptrs))
    m = gms.gms_manifest_build(entries, w.image_bytes)
    bd = torch.zeros(m.n_blocks, dtype=torch.int64, device="cuda")
    td = torch.zeros(m.n_tensors, dtype=torch.int64, device="cuda")
    gms.gms_restore(m, image, gms.SRC_DEVICE, bd, td)
    gms.gms_manifest_set_expected(m, bd)
    torch.cuda.synchronize()
    assert np.array_equal(bd.cpu().numpy().view(np.uint64), obd) and np.array_equal(td.cpu().numpy().view(np.uint64), otd)
    gms.gms_service_commit(svc)

    # ---- device-preserving loss: the replacement attaches read-only and checks before it reuses
    cap = 32
    out = torch.zeros(2 * cap, dtype=torch.int64, device="cuda")
    cnt = torch.zeros(1, dtype=torch.int64, device="cuda")
    per_tensor = torch.zeros(m.n_tensors, dtype=torch.int32, device="cuda")

    def check():
        gms.gms_digest(m, bd, td)
        gms.gms_verify(m, bd, out, cap, cnt)
        gms.gms_verify_tensors(m, bd, per_tensor)
        torch.cuda.synchronize()
        n = int(cnt.item())
        pairs = out.cpu().numpy().view(np.uint64).reshape(cap, 2)[: min(n, cap)]
        return n, [(int(a), int(b)) for a, b in pairs]

    gms.gms_service_acquire_ro(svc)
    assert check() == (0, [])  # intact: reuse, nothing to move
    gms.gms_service_release_ro(svc)

    # ---- the state is damaged while a writer holds it (host-made single-bit flips in three tensors)
    gms.gms_service_acquire_rw(svc)
    flips = W.flip_positions(w, 3, seed=303)
    for row, byte, bit in flips:
        addr = ptrs[row] + byte
        cell = torch.zeros(1, dtype=torch.uint8, device="cuda")
        view = _byte_view(addr)  # a 1-byte read-modify-write through torch
        cell.copy_(view)
        view.copy_(cell ^ (1 << bit))
    torch.cuda.synchronize()
    gms.gms_service_commit(svc)

    gms.gms_service_acquire_ro(svc)
    n, pairs = check()
    want_pairs = sorted((int(w.rows[r]["tensor_id"]), b // 4096) for r, b, _ in flips)
    assert n == 3 and sorted(pairs) == want_pairs
    # order of the list is (entry position, block)
    pos = {int(r["tensor_id"]): i for i, r in enumerate(w.rows)}
    assert pairs == sorted(pairs, key=lambda tb: (pos[tb[0]], tb[1]))
    counts = per_tensor.cpu().numpy()
    assert counts.sum() == 3 and all(counts[pos[t]] >= 1 for t, _ in pairs)
    gms.gms_service_release_ro(svc)

    # ---- repair only what is damaged: a manifest of the damaged entries, same image, same addresses
    gms.gms_service_acquire_rw(svc)
    damaged = sorted({pos[t] for t, _ in pairs})
    sub = gms.gms_manifest_build(entries[damaged], w.image_bytes)
    sub_bd = torch.zeros(sub.n_blocks, dtype=torch.int64, device="cuda")
    sub_td = torch.zeros(sub.n_tensors, dtype=torch.int64, device="cuda")
    gms.gms_restore(sub, image, gms.SRC_DEVICE, sub_bd, sub_td)
    torch.cuda.synchronize()
    assert sub.payload_bytes == sum(int(w.rows[i]["nbytes"]) for i in damaged) < w.payload_bytes
    assert np.array_equal(sub_td.cpu().numpy().view(np.uint64), otd[damaged])  # the repaired tensors digest as the oracle says
    gms.gms_service_commit(svc)
    gms.gms_service_acquire_ro(svc)
    assert check() == (0, [])  # the whole state is intact again
    assert np.array_equal(td.cpu().numpy().view(np.uint64), otd)
    gms.gms_service_release_ro(svc)
    sub.close()
    m.close()
    svc.close()


def _byte_view(addr: int):
    """A 1-element uint8 tensor over a device address (DLPack-free: through the CUDA array interface)."""

    class _Holder:
        __cuda_array_interface__ = {"shape": (1,), "typestr": "|u1", "data": (int(addr), False), "version": 3}

    return torch.as_tensor(_Holder(), device="cuda")
