"""Writes tests/golden/oracle_regression.txt: digests the CPU oracle produces today for a few fixed inputs.

    python tests/golden/make_oracle_regression.py

The file is a drift alarm for the oracle itself, not a pin of its correctness (the pins are the published
SplitMix64 values, closed forms and brute-force checks in tests/test_oracle_pins.py): once written, any later
change to the oracle's arithmetic shows up as a difference in tests/test_oracle_pins.py.  This script calls
nothing but the oracle; the inputs come from the explicit 64-bit LCG below (Knuth's MMIX constants), so they do
not depend on any library's random generator.
"""
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

from oracle import gms_oracle as oracle  # noqa: E402

OUT = os.path.join(HERE, "oracle_regression.txt")


def lcg_bytes(n: int, seed: int) -> np.ndarray:
    """n bytes: the top byte of successive states of x <- x * 6364136223846793005 + 1442695040888963407 (mod 2^64)."""
    out = np.empty(n, np.uint8)
    x = seed & (2**64 - 1)
    for i in range(n):
        x = (x * 6364136223846793005 + 1442695040888963407) & (2**64 - 1)
        out[i] = x >> 56
    return out


def cases():
    """Yields (name, list of uint64 values)."""
    # a record with a zero-length tensor, a one-byte tensor, an exact block, ragged tails and a shared source
    rows = [(11, 0, 4096, 10000), (12, 10000, 0, 0), (13, 10000, 16384, 1), (14, 10016, 20480, 4096),
            (15, 14112, 28672, 12289), (16, 0, 45056, 777)]
    rec = oracle.make_record(rows)
    image = lcg_bytes(26416, 1)
    slab = np.zeros(49152, np.uint8)
    rc, bd, td = oracle.restore(rec, image, slab)
    assert rc == 0
    yield "restore.block_digests", bd
    yield "restore.tensor_digests", td
    slab[4096 + 4500] ^= 0x40   # tensor 11, block 1
    slab[28672 + 12288] ^= 0x01  # tensor 15, block 3 (its one-byte tail)
    rc, bd2, td2 = oracle.digest(rec, slab)
    assert rc == 0
    yield "digest_after_two_flips.tensor_digests", td2
    count, mm = oracle.verify(rec, bd2, bd, cap=8)
    yield "verify.count_then_pairs", [count] + [int(v) for m in mm for v in (m["tensor_id"], m["block"])]
    # KV: 3 planes x 7 blocks of 8 KiB, ids with two out of range
    n_planes, n_blocks, bb = 3, 7, 8192
    ids = np.array([6, -1, 2, 7, 0], np.int32)
    pool = lcg_bytes(n_planes * n_blocks * bb, 2)
    img = lcg_bytes(n_planes * len(ids) * bb, 3)
    rc, kbd, kkd, skipped = oracle.kv_restore(pool, n_blocks * bb, bb, n_planes, n_blocks, bb, img, len(ids) * bb, bb, ids)
    assert rc == 0
    yield "kv_restore.kv_digests_then_skipped", list(kkd) + [skipped]
    yield "kv_restore.block_digests_xor", [int(np.bitwise_xor.reduce(kbd))]
    rc, kbd2, kkd2, _ = oracle.kv_digest(pool, n_blocks * bb, bb, n_planes, n_blocks, bb, np.array([1, 3, 5], np.int32))
    assert rc == 0
    yield "kv_digest.kv_digests", kkd2


def render() -> str:
    lines = ["# written by tests/golden/make_oracle_regression.py (calls only oracle/); do not edit by hand"]
    for name, values in cases():
        lines.append(name + " " + " ".join(f"{int(v):016X}" for v in values))
    return "\n".join(lines) + "\n"


if __name__ == "__main__":
    with open(OUT, "w") as f:
        f.write(render())
    print("wrote", OUT)
