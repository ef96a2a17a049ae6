"""The service's memory across processes (Section 4, GMS paragraph: the service keeps the creator handles and passes
file descriptors over Unix sockets; Section 3.2: the state outlives the engine that filled it and the replacement
attaches it read-only and checks that it is intact).

This process is the service: it creates shareable slabs, runs the ownership protocol and exports the slabs.  Every
client is a separate process (tests/service_client.py) that gets the descriptors over a socket pair:
a writer that restores an image into the allocations and then disappears without cleaning up, a reader that finds
the contents intact (digests equal to the oracle's restore of the same image, nothing to report, bytes identical), a
second writer that flips bytes, and a reader that names exactly the blocks the oracle's verify names.  No process
ever writes through a read-only mapping, and a client only leaves with none of its work in flight."""
import hashlib
import json
import os
import socket
import struct
import subprocess
import sys

import numpy as np
import pytest

from paper_2609_25451_b200 import gms
from paper_2609_25451_b200 import workloads as W

MiB = 1 << 20
HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)


def run_client(job, fds, expect_exit=0):
    """Starts a client process, hands it the job and the descriptors, returns its reply."""
    ours, theirs = socket.socketpair(socket.AF_UNIX, socket.SOCK_STREAM)
    ours.settimeout(300)
    env = dict(os.environ, PYTHONPATH=os.pathsep.join([ROOT, HERE, os.environ.get("PYTHONPATH", "")]))
    proc = subprocess.Popen([sys.executable, os.path.join(HERE, "service_client.py"), str(theirs.fileno())],
                            pass_fds=[theirs.fileno()], env=env, cwd=ROOT)
    theirs.close()
    try:
        data = json.dumps(job).encode()
        socket.send_fds(ours, [struct.pack("<II", len(data), len(fds))], fds)
        ours.sendall(data)
        head = b""
        while len(head) < 4:
            part = ours.recv(4 - len(head))
            assert part, "the client closed the socket without a reply"
            head += part
        (n,) = struct.unpack("<I", head)
        body = b""
        while len(body) < n:
            part = ours.recv(n - len(body))
            assert part
            body += part
        assert proc.wait(timeout=120) == expect_exit
        return json.loads(body.decode())
    finally:
        ours.close()
        if proc.poll() is None:
            proc.kill()  # the exact child started above
            proc.wait()


def export_all(svc, n_slabs):
    return [gms.gms_service_export_fd(svc, k) for k in range(n_slabs)]


def test_export_needs_a_shareable_service():
    s = gms.gms_service_create(8 * MiB, gms.SERVICE_DRY_RUN)
    gms.gms_service_acquire_rw(s)
    p = gms.gms_service_alloc(s, 1000)
    info = gms.gms_service_slab(s, 0)
    assert info["address"] == p and info["bytes"] == 8 * MiB and info["dedicated"] == 0
    with pytest.raises(gms.GmsError) as ei:
        gms.gms_service_slab(s, 1)
    assert ei.value.status == gms.ERR_RANGE
    with pytest.raises(gms.GmsError) as ei:
        gms.gms_service_export_fd(s, 0)  # a dry run has nothing to export
    assert ei.value.status == gms.ERR_STATE
    with pytest.raises(gms.GmsError) as ei:
        gms.gms_service_export_fd(s, 5)
    assert ei.value.status == gms.ERR_RANGE
    s.close()
    import ctypes

    L = gms.lib()
    assert L.gms_import_create(None, None, 1, 0, None) == gms.ERR_NULL
    assert L.gms_import_destroy(None) == gms.OK
    assert L.gms_import_address(None, 0, None) == gms.ERR_NULL
    assert L.gms_service_slab(None, 0, None) == gms.ERR_NULL
    assert L.gms_service_export_fd(None, 0, None) == gms.ERR_NULL
    out = ctypes.c_void_p()
    assert L.gms_service_create(0, 4, ctypes.byref(out)) == gms.ERR_ARG  # unknown flag


@pytest.mark.gpu
def test_state_survives_its_writer_and_is_checked_by_another_process(oracle):
    from gpu_harness import oracle_record

    w = W.mixed_manifest(n_small=400, n_large=3, large_bytes=(6 * MiB) + 40, round16=False, seed=301)
    seed = 302
    image_h = W.random_bytes_host(w.image_bytes, seed=seed)
    rec = oracle_record(oracle, w)
    slab_h = np.zeros(w.slab_bytes, np.uint8)
    rc, obd, otd = oracle.restore(rec, image_h, slab_h)
    assert rc == 0

    # a service without the flag cannot export
    plain = gms.gms_service_create(8 * MiB)
    gms.gms_service_acquire_rw(plain)
    gms.gms_service_alloc(plain, 1000)
    with pytest.raises(gms.GmsError) as ei:
        gms.gms_service_export_fd(plain, 0)
    assert ei.value.status == gms.ERR_STATE
    gms.gms_service_abort(plain)
    plain.close()

    svc = gms.gms_service_create(8 * MiB, gms.SERVICE_SHAREABLE)
    gms.gms_service_acquire_rw(svc)
    ptrs = [gms.gms_service_alloc(svc, max(1, int(r["nbytes"]))) for r in w.rows]
    n_slabs = gms.gms_service_info(svc)["n_slabs"]
    assert n_slabs >= 3
    slabs = [gms.gms_service_slab(svc, k) for k in range(n_slabs)]

    def place(p):
        for k, s in enumerate(slabs):
            if s["address"] <= p < s["address"] + s["bytes"]:
                return k, p - s["address"]
        raise AssertionError("allocation outside every slab")

    rows = [[int(r["tensor_id"]), int(r["src_offset"]), *place(p), int(r["nbytes"])] for r, p in zip(w.rows, ptrs)]
    job = {"slabs": slabs, "rows": rows, "image_bytes": int(w.image_bytes)}
    try:
        # ---- RW: the writer fills the allocations and is gone (exit code 17, nothing cleaned up)
        fds = export_all(svc, n_slabs)
        rep = run_client(dict(job, role="writer", seed=seed), fds, expect_exit=17)
        for fd in fds:
            os.close(fd)
        assert rep["status"] == 0
        assert np.array_equal(np.frombuffer(bytes.fromhex(rep["bd"]), np.uint64), obd)
        assert np.array_equal(np.frombuffer(bytes.fromhex(rep["td"]), np.uint64), otd)
        recorded = rep["bd"]
        gms.gms_service_commit(svc)

        # ---- RO: another process attaches what survived and finds it intact
        gms.gms_service_acquire_ro(svc)
        fds = export_all(svc, n_slabs)
        rep = run_client(dict(job, role="reader", expected=recorded, cap=8, remap_in_place=True), fds)
        for fd in fds:
            os.close(fd)
        want = hashlib.sha256()
        for r in w.rows:
            s0, n = int(r["src_offset"]), int(r["nbytes"])
            want.update(image_h[s0:s0 + n].tobytes())
        assert rep["status"] == 0  # (a fresh process need not get the service's addresses: rep["same"] may be False)
        assert rep["count"] == 0 and rep["pairs"] == []
        assert rep["bd"] == recorded and np.array_equal(np.frombuffer(bytes.fromhex(rep["td"]), np.uint64), otd)
        assert rep["sha256"] == want.hexdigest(), "the bytes a second process reads are not the bytes the writer put there"
        gms.gms_service_release_ro(svc)

        # ---- RW again: a writer damages three bytes in two tensors; the next reader names exactly those blocks
        gms.gms_service_acquire_rw(svc)
        big = [k for k, r in enumerate(w.rows) if int(r["nbytes"]) > 3 * 4096]
        flips = [[big[0], 5, 3], [big[0], 2 * 4096 + 77, 0], [big[-1], int(w.rows[big[-1]]["nbytes"]) - 1, 7]]
        fds = export_all(svc, n_slabs)
        rep = run_client(dict(job, role="damager", flips=flips), fds)
        for fd in fds:
            os.close(fd)
        assert rep["status"] == 0
        gms.gms_service_commit(svc)
        gms.gms_service_acquire_ro(svc)
        for row, byte, bit in flips:
            slab_h[int(w.rows[row]["dst_offset"]) + byte] ^= 1 << bit
        rc, dbd, dtd = oracle.digest(rec, slab_h)
        ocount, omm = oracle.verify(rec, dbd, obd, 8)
        assert rc == 0 and ocount == 3
        fds = export_all(svc, n_slabs)
        rep = run_client(dict(job, role="reader", expected=recorded, cap=8), fds)
        for fd in fds:
            os.close(fd)
        assert rep["status"] == 0 and rep["count"] == ocount
        assert [tuple(p) for p in rep["pairs"]] == [(int(a), int(b)) for a, b in omm]
        assert np.array_equal(np.frombuffer(bytes.fromhex(rep["bd"]), np.uint64), dbd)
        assert np.array_equal(np.frombuffer(bytes.fromhex(rep["td"]), np.uint64), dtd)
        gms.gms_service_release_ro(svc)
    finally:
        svc.close()
