"""Helpers for the GPU parity tests: put a workload on the device, call the C ABI through the
binding, bring results back as numpy arrays, and build the oracle's view of the same inputs."""
from __future__ import annotations

import numpy as np
import torch

from paper_2609_25451_b200 import gms

CANARY = 0x5A5A5A5A5A5A5A5A
PAD = 32  # canary words on both sides of every output array
FILL = 0xEE  # untouched slab bytes


def oracle_record(oracle, w):
    return oracle.make_record((r["tensor_id"], r["src_offset"], r["dst_offset"], r["nbytes"]) for r in w.rows)


def guarded_u64(n: int) -> torch.Tensor:
    return torch.full((n + 2 * PAD,), CANARY, dtype=torch.int64, device="cuda")


def payload_of(t: torch.Tensor, n: int) -> np.ndarray:
    """Host copy of the n payload words; asserts both canary bands are intact."""
    h = t.cpu().numpy().view(np.uint64)
    assert (h[:PAD] == CANARY).all() and (h[PAD + n:] == CANARY).all(), "output array was written out of bounds"
    return h[PAD:PAD + n].copy()


class DeviceWorkload:
    """A workload resident on cuda:0: image, destination slab, manifest and guarded outputs."""

    def __init__(self, w, image_host: np.ndarray | None = None, image_dev: torch.Tensor | None = None,
                 slab: torch.Tensor | None = None):
        self.w = w
        if image_dev is None:
            image_dev = torch.from_numpy(np.ascontiguousarray(image_host)).cuda()
        self.image = image_dev
        self.slab = slab if slab is not None else torch.full((w.slab_bytes,), FILL, dtype=torch.uint8, device="cuda")
        base = self.slab.data_ptr()
        assert base % 16 == 0 and self.image.data_ptr() % 16 == 0
        self.entries = gms.make_entries(
            (r["tensor_id"], r["src_offset"], base + int(r["dst_offset"]), r["nbytes"]) for r in w.rows)
        self.m = gms.gms_manifest_build(self.entries, w.image_bytes)
        self.nb, self.nt = self.m.n_blocks, self.m.n_tensors
        self.bd = guarded_u64(self.nb)
        self.td = guarded_u64(self.nt)

    def bd_ptr(self):
        return self.bd.data_ptr() + 8 * PAD

    def td_ptr(self):
        return self.td.data_ptr() + 8 * PAD

    def reset_outputs(self):
        self.bd.fill_(CANARY)
        self.td.fill_(CANARY)

    def restore(self, image=None, kind=gms.SRC_DEVICE, want_bd=True, want_td=True):
        self.reset_outputs()
        gms.gms_restore(self.m, self.image if image is None else image, kind, self.bd_ptr() if want_bd else None,
                        self.td_ptr() if want_td else None)
        torch.cuda.synchronize()
        assert gms.gms_last_device_status(self.m) == 0
        return payload_of(self.bd, self.nb), payload_of(self.td, self.nt)

    def digest(self, want_bd=True, want_td=True):
        self.reset_outputs()
        gms.gms_digest(self.m, self.bd_ptr() if want_bd else None, self.td_ptr() if want_td else None)
        torch.cuda.synchronize()
        assert gms.gms_last_device_status(self.m) == 0
        return payload_of(self.bd, self.nb), payload_of(self.td, self.nt)

    def verify(self, cap: int):
        out = torch.full((2 * cap + 2 * PAD,), CANARY, dtype=torch.int64, device="cuda")
        cnt = guarded_u64(1)
        gms.gms_verify(self.m, self.bd_ptr(), out.data_ptr() + 8 * PAD, cap, cnt.data_ptr() + 8 * PAD)
        torch.cuda.synchronize()
        count = int(payload_of(cnt, 1)[0])
        pairs = payload_of(out, 2 * cap).reshape(cap, 2)
        k = min(count, cap)
        assert (pairs[k:] == CANARY).all(), "verify wrote past min(count, cap)"
        return count, [(int(a), int(b)) for a, b in pairs[:k]]

    def fused(self, cap: int, restore: bool = False):
        """gms_digest_verify (or gms_restore_verify from the device image): digests, count and mismatch pairs."""
        self.reset_outputs()
        out = torch.full((2 * cap + 2 * PAD,), CANARY, dtype=torch.int64, device="cuda")
        cnt = guarded_u64(1)
        if restore:
            gms.gms_restore_verify(self.m, self.image, gms.SRC_DEVICE, self.bd_ptr(), self.td_ptr(), out.data_ptr() + 8 * PAD, cap,
                                   cnt.data_ptr() + 8 * PAD)
        else:
            gms.gms_digest_verify(self.m, self.bd_ptr(), self.td_ptr(), out.data_ptr() + 8 * PAD, cap, cnt.data_ptr() + 8 * PAD)
        torch.cuda.synchronize()
        assert gms.gms_last_device_status(self.m) == 0
        count = int(payload_of(cnt, 1)[0])
        pairs = payload_of(out, 2 * cap).reshape(cap, 2)
        k = min(count, cap)
        assert (pairs[k:] == CANARY).all(), "the fused verify wrote past min(count, cap)"
        return payload_of(self.bd, self.nb), payload_of(self.td, self.nt), count, [(int(a), int(b)) for a, b in pairs[:k]]

    def slab_host(self) -> np.ndarray:
        return self.slab.cpu().numpy()

    def flip(self, row: int, byte: int, bit: int):
        """Host-made corruption: one bit of one destination byte, via a 1-byte read-modify-write."""
        pos = int(self.w.rows[row]["dst_offset"]) + byte
        v = int(self.slab[pos].item())
        self.slab[pos] = v ^ (1 << bit)

    def close(self):
        self.m.close()
