"""The oracle over a whole full-size workload in a few seconds: one Python thread per host core, each calling the
unchanged single-threaded oracle on whole tensors (or whole KV slots) -- ctypes releases the interpreter lock while
the C code runs.  Nothing here computes a digest; it only deals the oracle's own calls out to threads and puts the
results where the record order says they belong."""
from __future__ import annotations

import concurrent.futures as cf
import os

import numpy as np


def all_digests(oracle, rec, fetch, threads: int | None = None):
    """Block and tensor digests of every entry of `rec`, from the oracle.

    fetch(t) returns the bytes entry t is (or should be) made of, as a contiguous uint8 array.
    Returns (block_digests in record order, tensor_digests)."""
    base, total = oracle.block_bases(rec)
    bd = np.zeros(total, dtype=np.uint64)
    td = np.zeros(len(rec), dtype=np.uint64)

    def one(t):
        T, d = oracle.tensor_digest(fetch(t))
        bd[int(base[t]):int(base[t]) + d.size] = d
        td[t] = T

    order = sorted(range(len(rec)), key=lambda t: -int(rec[t]["nbytes"]))  # largest first: the pool balances the rest
    with cf.ThreadPoolExecutor(threads or os.cpu_count() or 1) as ex:
        list(ex.map(one, order))
    return bd, td


def all_kv_digests(oracle, n_sel: int, n_planes: int, block_bytes: int, fetch_slot, threads: int | None = None):
    """Block digests [j][plane][sub-block] and KV digests of every list position j, from the oracle: a slot's KV
    digest is the tensor digest of its planes concatenated in plane order, and its block digests are that tensor's.

    fetch_slot(j) returns the slot's planes as one contiguous uint8 array of n_planes * block_bytes bytes."""
    per = n_planes * (block_bytes // 4096)
    bd = np.zeros(n_sel * per, dtype=np.uint64)
    kd = np.zeros(n_sel, dtype=np.uint64)

    def one(j):
        T, d = oracle.tensor_digest(fetch_slot(j))
        assert d.size == per
        bd[j * per:(j + 1) * per] = d
        kd[j] = T

    with cf.ThreadPoolExecutor(threads or os.cpu_count() or 1) as ex:
        list(ex.map(one, range(n_sel)))
    return bd, kd
