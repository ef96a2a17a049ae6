"""A client process of a gms_service that lives in another process (run by tests/test_gpu_service_process.py).

It is started with one end of a Unix socket pair, receives a job (a JSON header plus the slabs' file descriptors,
sent with SCM_RIGHTS), maps the slabs with gms_import_create and plays one of three parts:

  writer   imports the slabs writable, restores a seeded image into the allocations, reports the digests and then
           leaves WITHOUT any clean-up (os._exit), the way a crashed engine would: its mappings go with the process,
           the memory stays with the service
  reader   imports read-only, digests and verifies the allocations in place against the recorded digests
           (gms_digest_verify), captures them into a packed image and reports count, pairs, digests and a hash
  damager  imports writable and flips single bytes (captured, changed and restored through 16-byte entries)

Only the library's C ABI touches the imported memory; torch provides this process's own buffers."""
import hashlib
import json
import os
import socket
import struct
import sys

import numpy as np


def recv_exact(sock, n):
    buf = b""
    while len(buf) < n:
        part = sock.recv(n - len(buf))
        if not part:
            raise EOFError("the other side closed the socket")
        buf += part
    return buf


def recv_job(sock):
    """Header length (u32), number of descriptors (u32), then the JSON header; the descriptors ride on the first bytes."""
    msg, fds, _, _ = socket.recv_fds(sock, 8, 64)
    assert len(msg) == 8
    n_json, n_fds = struct.unpack("<II", msg)
    assert len(fds) == n_fds
    return json.loads(recv_exact(sock, n_json).decode()), fds


def send_reply(sock, obj):
    data = json.dumps(obj).encode()
    sock.sendall(struct.pack("<I", len(data)) + data)


def main():
    sock = socket.socket(fileno=int(sys.argv[1]))
    sock.settimeout(300)
    job, fds = recv_job(sock)

    import torch

    from paper_2609_25451_b200 import gms
    from paper_2609_25451_b200 import workloads as W

    role = job["role"]
    flags = (gms.IMPORT_WRITABLE if role in ("writer", "damager") else 0) | (gms.IMPORT_SAME_ADDRESS if job.get("same_address") else 0)
    imp = gms.gms_import_create(fds, job["slabs"], flags)
    base = [imp.address(k) for k in range(len(fds))]
    if job.get("remap_in_place"):
        # the addresses of a mapping that has just been dropped are free: asking for exactly those must succeed, and
        # asking for them while they are still mapped must be refused (GMS_ERR_RANGE), not answered with other addresses
        mine = [dict(s, address=b) for s, b in zip(job["slabs"], base)]
        try:
            gms.gms_import_create(fds, mine, flags | gms.IMPORT_SAME_ADDRESS)
            refused = False
        except gms.GmsError as e:
            refused = e.status == gms.ERR_RANGE
        imp.close()
        imp = gms.gms_import_create(fds, mine, flags | gms.IMPORT_SAME_ADDRESS)
        assert refused and [imp.address(k) for k in range(len(fds))] == base
    for fd in fds:
        os.close(fd)  # the import holds its own references
    same = all(b == s["address"] for b, s in zip(base, job["slabs"]))
    rows = job["rows"]  # [tensor_id, src_offset, slab, offset in the slab, nbytes]
    ent = gms.make_entries((r[0], r[1], base[r[2]] + r[3], r[4]) for r in rows)
    m = gms.gms_manifest_build(ent, job["image_bytes"])
    bd = torch.zeros(max(m.n_blocks, 1), dtype=torch.int64, device="cuda")
    td = torch.zeros(max(m.n_tensors, 1), dtype=torch.int64, device="cuda")
    hexof = lambda t, n: t[:n].cpu().numpy().tobytes().hex()

    if role == "writer":
        image = torch.from_numpy(W.random_bytes_host(job["image_bytes"], seed=job["seed"])).cuda()
        gms.gms_restore(m, image, gms.SRC_DEVICE, bd, td)
        torch.cuda.synchronize()
        send_reply(sock, {"status": gms.gms_last_device_status(m), "bd": hexof(bd, m.n_blocks), "td": hexof(td, m.n_tensors), "same": same})
        sock.close()
        os._exit(17)  # no gms_import_destroy, no context tear-down of our own: the process just goes

    if role == "reader":
        exp = torch.from_numpy(np.frombuffer(bytes.fromhex(job["expected"]), dtype=np.int64).copy()).cuda()
        gms.gms_manifest_set_expected(m, exp)
        cap = job["cap"]
        out = torch.zeros(2 * cap, dtype=torch.int64, device="cuda")
        cnt = torch.full((1,), -1, dtype=torch.int64, device="cuda")
        gms.gms_digest_verify(m, bd, td, out, cap, cnt)
        back = torch.zeros(job["image_bytes"], dtype=torch.uint8, device="cuda")
        gms.gms_capture(m, back, gms.SRC_DEVICE, None, None)
        torch.cuda.synchronize()
        h = hashlib.sha256()
        back_h = back.cpu().numpy()
        for r in rows:
            h.update(back_h[r[1]:r[1] + r[4]].tobytes())
        count = int(cnt.item())
        pairs = out.cpu().numpy().view(np.uint64).reshape(cap, 2)[:min(count, cap)].tolist()
        send_reply(sock, {"status": gms.gms_last_device_status(m), "count": count, "pairs": pairs, "bd": hexof(bd, m.n_blocks),
                          "td": hexof(td, m.n_tensors), "sha256": h.hexdigest(), "same": same})
    elif role == "damager":
        for row, byte, bit in job["flips"]:
            addr = base[rows[row][2]] + rows[row][3] + (byte & ~15)
            one = gms.gms_manifest_build(gms.make_entries([(1, 0, addr, 16)]), 16)
            cell = torch.zeros(16, dtype=torch.uint8, device="cuda")
            gms.gms_capture(one, cell, gms.SRC_DEVICE, None, None)
            torch.cuda.synchronize()
            cell[byte & 15] ^= (1 << bit)
            gms.gms_restore(one, cell, gms.SRC_DEVICE, None, None)
            torch.cuda.synchronize()
            one.close()
        send_reply(sock, {"status": 0, "same": same})
    m.close()
    imp.close()
    sock.close()


if __name__ == "__main__":
    main()
