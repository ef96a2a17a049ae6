"""gms_verify_flat_noalloc: the verify step for callers that cannot allocate device memory
(a checker on a GPU whose memory is already fully handed out, or a watchdog that must stay out
of the allocator while an engine serves).  The entry point keeps its working tables in a fixed
array inside the library, so the checks that matter are: it reports exactly what gms_verify
reports for a one-tensor manifest; a second call right after the first is not confused by what
the first left in the shared array (different size, different corruption); and sizes beyond the
fixed capacity are refused on the host.  Inputs above 16,384 digest slots take the path that really
uses the array (per-segment counters written by one kernel and read by the next), so those cases
put differences on both sides of segment boundaries, in the first and last slot, in a run longer
than a segment and in the ragged last segment, up to the entry point's maximum size, and compare
with the CPU oracle's verify of a one-entry record.  This file is collected last on purpose."""
import ctypes

import numpy as np
import pytest

torch = pytest.importorskip("torch")

from paper_2609_25451_b200 import gms  # noqa: E402
from paper_2609_25451_b200 import workloads as W  # noqa: E402


def test_sizes_beyond_the_fixed_capacity_are_refused_on_the_host():
    # no GPU needed: the size check precedes any CUDA call
    fake = ctypes.c_void_p(0x7F0000000000)
    rc = gms.lib().gms_verify_flat_noalloc(fake, fake, gms.NOALLOC_MAX_BLOCKS + 1, 7, fake, 4, fake, None)
    assert rc == gms.ERR_TOO_LARGE
    assert "capacity" in gms.gms_strerror(rc)
    assert gms.lib().gms_verify_flat_noalloc(None, None, 5, 7, None, 0, None, None) == gms.ERR_NULL


def _both_verifies(nbytes, tensor_id, corrupt_blocks, cap, seed):
    """Restore one tensor, record its digests, corrupt some blocks (host-made), digest again, and
    return what gms_verify and gms_verify_flat_noalloc each report."""
    w = W.pack_layout("flat", [nbytes], seed=seed, id_base=tensor_id)
    w.rows["tensor_id"] = tensor_id
    image = torch.from_numpy(W.random_bytes_host(w.image_bytes, seed=seed)).cuda()
    slab = torch.zeros(w.slab_bytes, dtype=torch.uint8, device="cuda")
    off = int(w.rows[0]["dst_offset"])
    ent = gms.make_entries([(tensor_id, 0, slab.data_ptr() + off, nbytes)])
    m = gms.gms_manifest_build(ent, w.image_bytes)
    nb = m.n_blocks
    bd = torch.zeros(nb, dtype=torch.int64, device="cuda")
    gms.gms_restore(m, image, gms.SRC_DEVICE, bd, None)
    gms.gms_manifest_set_expected(m, bd)
    expected = bd.clone()  # the caller's own copy of the digests recorded at commit
    for b in corrupt_blocks:
        pos = off + min(nbytes - 1, b * 4096 + 17)
        slab[pos] = int(slab[pos].item()) ^ 0x04
    gms.gms_digest(m, bd, None)

    def run(fn):
        out = torch.full((2 * cap + 8,), -1, dtype=torch.int64, device="cuda")
        cnt = torch.full((1,), -1, dtype=torch.int64, device="cuda")
        fn(out, cnt)
        torch.cuda.synchronize()
        k = min(int(cnt.item()), cap)
        assert (out[2 * k:] == -1).all()
        return int(cnt.item()), out[: 2 * k].cpu().numpy().view(np.uint64).reshape(-1, 2).tolist()

    old = run(lambda out, cnt: gms.gms_verify(m, bd, out, cap, cnt))
    new = run(lambda out, cnt: gms.gms_verify_flat_noalloc(bd, expected, nb, tensor_id, out, cap, cnt))
    m.close()
    return old, new, nb


@pytest.mark.gpu
def test_flat_noalloc_verify_matches_gms_verify_on_two_calls_in_a_row():
    # integer outputs: the comparison is exact, as in every other parity test of this suite
    first = sorted({0, 1, 2047, 2048, 2049, 4095, 4096, 9000, 12287} | set(range(5000, 5040)))
    old, new, nb = _both_verifies(4096 * 12288, tensor_id=4242, corrupt_blocks=first, cap=64, seed=3)
    assert nb == 12288 and old[0] == len(first)
    assert new == old
    assert [b for _, b in new[1]] == first[: len(new[1])] and all(t == 4242 for t, _ in new[1])
    # second call straight after: smaller tensor, other blocks, cap below the count, ragged last block
    second = [3, 700, 701, 2500]
    old2, new2, nb2 = _both_verifies(4096 * 2500 + 100, tensor_id=99, corrupt_blocks=second, cap=3, seed=4)
    assert nb2 == 2501 and old2[0] == 4 and len(old2[1]) == 3
    assert new2 == old2
    # and a clean comparison reports nothing, even though the array still holds the last call's counts
    old3, new3, _ = _both_verifies(4096 * 300, tensor_id=5, corrupt_blocks=[], cap=8, seed=5)
    assert old3 == (0, []) and new3 == old3


def _flat_case(oracle, n_blocks, bad_slots, cap, tensor_id, seed):
    """Two plain device arrays of n_blocks words that differ exactly in bad_slots; returns what the entry point
    reported and what the oracle's verify of a one-entry record says for the same arrays."""
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    expected = torch.randint(-(2**63), 2**63 - 1, (n_blocks,), dtype=torch.int64, device="cuda", generator=g)
    computed = expected.clone()
    idx = torch.tensor(sorted(bad_slots), dtype=torch.int64, device="cuda")
    if len(bad_slots):
        computed[idx] ^= 0x4000
    out = torch.full((2 * cap + 8,), -1, dtype=torch.int64, device="cuda")
    cnt = torch.full((1,), -1, dtype=torch.int64, device="cuda")
    gms.gms_verify_flat_noalloc(computed, expected, n_blocks, tensor_id, out, cap, cnt)
    torch.cuda.synchronize()
    count = int(cnt.item())
    k = min(count, cap)
    assert (out[2 * k:] == -1).all(), "wrote past min(count, cap)"
    got = out[: 2 * k].cpu().numpy().view(np.uint64).reshape(-1, 2).tolist()
    rec = oracle.make_record([(tensor_id, 0, 0, n_blocks * 4096)])
    ocount, omm = oracle.verify(rec, computed.cpu().numpy().view(np.uint64), expected.cpu().numpy().view(np.uint64), cap)
    want = [[int(m["tensor_id"]), int(m["block"])] for m in omm]
    return (count, got), (ocount, want)


@pytest.mark.gpu
@pytest.mark.parametrize("n_blocks", [70_000, gms.NOALLOC_MAX_BLOCKS])
def test_flat_noalloc_verify_on_the_segmented_path_against_the_oracle(oracle, n_blocks):
    seg = 2048
    last_seg0 = (n_blocks - 1) // seg * seg
    bad = {0, 1, seg - 1, seg, seg + 1, 5 * seg - 1, 5 * seg, 17 * seg + 1000, last_seg0 - 1, last_seg0, n_blocks - 1}
    bad |= set(range(9 * seg - 300, 10 * seg + 2500))  # a run longer than a segment, across two boundaries
    bad = {b for b in bad if 0 <= b < n_blocks}
    for cap in (len(bad) + 50, 7, 0):  # cap above and below the count
        got, want = _flat_case(oracle, n_blocks, bad, cap, tensor_id=31337, seed=n_blocks % 1000 + cap)
        assert got == want and got[0] == len(bad)
        assert [b for _, b in got[1]] == sorted(bad)[:cap]
    # straight after the large call: a smaller segmented call with other differences, then a one-CTA call, then a
    # clean segmented call -- the per-segment words the large call left behind must not leak into any of them
    got, want = _flat_case(oracle, 40_000, {3 * seg, 39_999}, 8, tensor_id=5, seed=77)
    assert got == want == (2, [[5, 3 * seg], [5, 39_999]])
    got, want = _flat_case(oracle, 300, {299}, 8, tensor_id=6, seed=78)
    assert got == want == (1, [[6, 299]])
    got, want = _flat_case(oracle, n_blocks, set(), 8, tensor_id=7, seed=79)
    assert got == want == (0, [])
