"""Seeded synthetic inputs for the tests and the benchmark.

This module holds layouts and random bytes only -- none of the method's
arithmetic (no digest, no copy logic) -- so that the CUDA library and the CPU
oracle can both be fed from it without sharing anything else.

A workload is a table of rows ``(tensor_id, src_offset, dst_offset, nbytes)``:
``src_offset`` addresses the packed snapshot image, ``dst_offset`` addresses one
destination slab from which the "device allocations" are carved in shuffled
order with guard bands between them (the slab mirrors a service that
suballocates tensors from a few large allocations).  Contents are uniformly
random bit patterns: bf16 weights are opaque 16-bit patterns to this path, so
random bits stand in for a real checkpoint (incompressible, NaN patterns
included).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

ROW_DTYPE = np.dtype([("tensor_id", "<u8"), ("src_offset", "<u8"), ("dst_offset", "<u8"), ("nbytes", "<u8")])
GUARD = 256  # bytes of untouched canary between neighbouring destinations
SEED_BASE = 0x25451000


@dataclass
class Workload:
    name: str
    rows: np.ndarray          # ROW_DTYPE
    image_bytes: int
    slab_bytes: int
    names: list = field(default_factory=list)

    @property
    def payload_bytes(self) -> int:
        return int(self.rows["nbytes"].sum())

    @property
    def n_blocks(self) -> int:
        return int(((self.rows["nbytes"] + 4095) // 4096).sum())


def _align16(x: int) -> int:
    return (x + 15) // 16 * 16


def pack_layout(name: str, sizes, *, seed: int, names=None, shuffle_dst: bool = True, id_base: int = 1000,
                guard: int = GUARD, image_bytes: int | None = None) -> Workload:
    """Packs tensors of the given byte sizes into an image (record order, 16-byte aligned
    offsets) and carves their destinations from one slab in a seeded shuffled order."""
    sizes = [int(s) for s in sizes]
    n = len(sizes)
    rng = np.random.default_rng(seed)
    rows = np.zeros(n, dtype=ROW_DTYPE)
    off = 0
    for t, s in enumerate(sizes):
        rows[t]["src_offset"] = off
        off += _align16(s)
    img = off if image_bytes is None else int(image_bytes)
    assert img >= off
    order = rng.permutation(n) if shuffle_dst else np.arange(n)
    off = guard
    for t in order:
        rows[t]["dst_offset"] = off
        off += _align16(sizes[t]) + guard
    ids = id_base + rng.permutation(n).astype(np.uint64) * 7  # distinct, unordered ids
    rows["tensor_id"] = ids
    rows["nbytes"] = sizes
    return Workload(name, rows, max(img, 16), max(off, 16), list(names) if names else [])


# ------------------------------------------------------------------ the five workload families
def tiny_manifest(seed: int = SEED_BASE + 1, n: int = 64) -> Workload:
    """64 tensors of 16*U{256..65536} bytes (4 KiB .. 1 MiB), about 32 MiB in all."""
    rng = np.random.default_rng(seed)
    sizes = 16 * rng.integers(256, 65536 + 1, size=n)
    return pack_layout("tiny-64", sizes, seed=seed + 100)


def llama_tensor_sizes(vocab_rows: int, hidden: int, inter: int, n_layers: int, q_rows: int, kv_rows: int,
                       final_norm: bool, elem: int = 2):
    """(name, bytes) of a Llama-style decoder in model order; q_rows/kv_rows are the
    projection output rows held by this rank."""
    out = [("embed", vocab_rows * hidden * elem)]
    for l in range(n_layers):
        out += [
            (f"l{l}.q", q_rows * hidden * elem), (f"l{l}.k", kv_rows * hidden * elem),
            (f"l{l}.v", kv_rows * hidden * elem), (f"l{l}.o", hidden * q_rows * elem),
            (f"l{l}.gate", inter * hidden * elem), (f"l{l}.up", inter * hidden * elem),
            (f"l{l}.down", hidden * inter * elem), (f"l{l}.norm1", hidden * elem), (f"l{l}.norm2", hidden * elem),
        ]
    if final_norm:
        out.append(("norm", hidden * elem))
    out.append(("lm_head", vocab_rows * hidden * elem))
    return out


def llama3_8b_manifest(seed: int = SEED_BASE + 2, shrink: int = 1) -> Workload:
    """Llama-3-8B weight shapes in bf16 (291 tensors, 16,060,522,496 bytes at shrink=1).
    ``shrink`` divides hidden-size-like dimensions to get a small manifest of the same structure."""
    ts = llama_tensor_sizes(128256 // shrink, 4096 // shrink, 14336 // shrink, 32, 4096 // shrink, 1024 // shrink, True)
    return pack_layout(f"llama3-8b/{shrink}", [s for _, s in ts], seed=seed, names=[n for n, _ in ts])


def llama3_70b_tp8_shard_manifest(seed: int = SEED_BASE + 5, shrink: int = 1, image_bytes: int | None = None) -> Workload:
    """One tensor-parallel-8 shard of Llama-3-70B in bf16 (722 tensors, 17,640,718,336 bytes at
    shrink=1).  With ``image_bytes`` set, the shard list is repeated (a second rank's shard) and cut
    at the last whole tensor that fits the image."""
    ts = llama_tensor_sizes(16032 // shrink, 8192 // shrink, 3584 // shrink, 80, 1024 // shrink, 128 // shrink, False)
    sizes, names = [s for _, s in ts], [n for n, _ in ts]
    if image_bytes is not None:
        all_sizes, all_names, used, rep, full = [], [], 0, 0, False
        while not full:
            for s, nm in zip(sizes, names):
                if used + _align16(s) > image_bytes:
                    full = True
                    break
                all_sizes.append(s)
                all_names.append(f"r{rep}.{nm}")
                used += _align16(s)
            rep += 1
        sizes, names = all_sizes, all_names
    return pack_layout(f"llama3-70b-tp8/{shrink}", sizes, seed=seed, names=names, image_bytes=image_bytes)


def mixed_manifest(seed: int = SEED_BASE + 4, n_small: int = 10000, n_large: int = 8, large_bytes: int = 256 << 20,
                   round16: bool = True, lo: int = 256, hi: int = 65536) -> Workload:
    """Launch-bound mix: n_small tensors with log-uniform sizes lo..hi bytes plus n_large big
    ones, interleaved in a seeded random order.  round16=False keeps the raw odd sizes."""
    rng = np.random.default_rng(seed)
    small = np.rint(np.exp(rng.uniform(math.log(lo), math.log(hi), size=n_small))).astype(np.int64)
    if round16:
        small = np.maximum(16, (small + 8) // 16 * 16)
    sizes = np.concatenate([small, np.full(n_large, large_bytes, dtype=np.int64)])
    sizes = sizes[rng.permutation(len(sizes))]
    return pack_layout(f"mixed-{n_small}+{n_large}", sizes, seed=seed + 100)


@dataclass
class KvWorkload:
    name: str
    n_planes: int        # layers x {K, V}
    n_blocks: int        # blocks per plane in the pool
    block_bytes: int     # tokens x kv_heads x head_dim x 2 bytes
    ids: np.ndarray      # int32, selected pool blocks, distinct, unsorted
    plane_stride: int
    block_stride: int
    img_plane_stride: int
    img_slot_stride: int

    @property
    def pool_bytes(self) -> int:
        return self.n_planes * self.plane_stride

    @property
    def image_bytes(self) -> int:
        return self.n_planes * self.img_plane_stride

    @property
    def payload_bytes(self) -> int:
        return len(self.ids) * self.n_planes * self.block_bytes


def kv_pool_workload(seed: int = SEED_BASE + 3, pool_bytes: float = 60e9, n_layers: int = 32, tokens: int = 16,
                     kv_heads: int = 8, head_dim: int = 128, fraction: float = 0.1) -> KvWorkload:
    """Paged KV pool for the 8B shape: 64 planes of 32 KiB blocks filling ``pool_bytes``; a
    seeded random ``fraction`` of the blocks (no repeats) is selected, in random order."""
    block_bytes = tokens * kv_heads * head_dim * 2
    n_planes = 2 * n_layers
    n_blocks = int(pool_bytes // (n_planes * block_bytes))
    n_sel = int(n_blocks * fraction)
    rng = np.random.default_rng(seed)
    ids = rng.permutation(n_blocks)[:n_sel].astype(np.int32)
    return KvWorkload(f"kv-{n_planes}x{n_blocks}x{block_bytes}", n_planes, n_blocks, block_bytes, ids,
                      plane_stride=n_blocks * block_bytes, block_stride=block_bytes,
                      img_plane_stride=max(n_sel, 1) * block_bytes, img_slot_stride=block_bytes)


# ------------------------------------------------------------------ contents
def random_bytes_host(nbytes: int, seed: int) -> np.ndarray:
    """Uniform random bytes on the host (numpy PCG64)."""
    rng = np.random.default_rng(seed)
    words = rng.integers(0, 2**64, size=(nbytes + 7) // 8, dtype=np.uint64)
    return words.view(np.uint8)[:nbytes].copy()


def fill_random_device(t, seed: int, chunk_bytes: int = 1 << 30):
    """Fills a uint8 torch tensor on a CUDA device with uniform random bits (seeded Philox),
    1 GiB at a time.  Returns the tensor."""
    import torch

    assert t.dtype == torch.uint8 and t.is_contiguous()
    g = torch.Generator(device=t.device)
    g.manual_seed(seed)
    n = t.numel()
    n8 = n // 8 * 8
    if n8:
        v = t[:n8].view(torch.int64)
        step = chunk_bytes // 8
        for a in range(0, v.numel(), step):
            b = min(v.numel(), a + step)
            v[a:b] = torch.randint(-(2**63), 2**63 - 1, (b - a,), dtype=torch.int64, device=t.device, generator=g)
    if n > n8:
        t[n8:] = torch.randint(0, 256, (n - n8,), dtype=torch.uint8, device=t.device, generator=g)
    return t


def flip_positions(w: Workload, n_flips: int, seed: int):
    """Seeded (row index, byte offset in tensor, bit) triples in distinct 4 KiB blocks of non-empty tensors."""
    rng = np.random.default_rng(seed)
    live = np.nonzero(w.rows["nbytes"] > 0)[0]
    out, seen = [], set()
    while len(out) < n_flips:
        t = int(rng.choice(live))
        byte = int(rng.integers(0, int(w.rows[t]["nbytes"])))
        if (t, byte // 4096) in seen:
            continue
        seen.add((t, byte // 4096))
        out.append((t, byte, int(rng.integers(0, 8))))
    return out
