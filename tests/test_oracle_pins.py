"""Pins for the CPU oracle: every check here compares the oracle with something
that does not come from the oracle -- published SplitMix64 outputs, values
evaluated independently from the definition (tests/golden/digest_pins.txt),
closed forms built from the textbook SplitMix64 *generator* (the stateful
form, not the oracle's multiply-by-index form), exhaustive single-bit flips,
and brute-force byte comparison.  A dropped term, a wrong shift or constant, a
wrong word/byte order or an off-by-one block/word index fails at least one.
"""
import os

import numpy as np
import pytest

G = 0x9E3779B97F4A7C15
M64 = (1 << 64) - 1
GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "digest_pins.txt")


def splitmix64_stream(seed, n):
    """Textbook SplitMix64 generator: state += G; output = finalizer(state)."""
    out, state = [], seed & M64
    for _ in range(n):
        state = (state + G) & M64
        z = state
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & M64
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & M64
        out.append(z ^ (z >> 31))
    return out


def load_golden():
    rows = {}
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, recipe, ds, t = [s.strip() for s in line.split("|")]
            rows[name] = ([int(x, 16) for x in ds.split(",") if x], int(t, 16) if t else None)
    return rows


GOLD = load_golden()


def words_le(words):
    return np.array([w & M64 for w in words], dtype="<u8").view(np.uint8)


RECIPES = {
    "zeros_4096": np.zeros(4096, np.uint8),
    "zeros_8192": np.zeros(8192, np.uint8),
    "one_byte_01": np.array([1], np.uint8),
    "eight_bytes_01": np.array([1, 0, 0, 0, 0, 0, 0, 0], np.uint8),
    "ff_4097": np.full(4097, 0xFF, np.uint8),
    "ramp7k3_10000": ((7 * np.arange(10000) + 3) & 0xFF).astype(np.uint8),
    "words_i_512": words_le(range(512)),
    "words_iG_512": words_le(i * G for i in range(512)),
}


def test_mix_matches_published_splitmix64_outputs(oracle):
    # published seed-0 outputs; mix(k*G) must equal the k-th output
    want = GOLD["splitmix64_seed0"][0]
    assert want == [16294208416658607535, 7960286522194355700, 487617019471545679, 17909611376780542444]
    assert [oracle.mix(k * G) for k in (1, 2, 3, 4)] == want
    assert oracle.mix(0) == 0


def test_mix_equals_textbook_generator_on_a_long_stream(oracle):
    stream = splitmix64_stream(0, 2000)
    assert [oracle.mix((k * G) & M64) for k in range(1, 2001)] == stream
    other = splitmix64_stream(0xDEADBEEFCAFEF00D, 64)
    assert [oracle.mix((0xDEADBEEFCAFEF00D + k * G) & M64) for k in range(1, 65)] == other


def test_mix_is_injective_on_a_sample(oracle):
    rng = np.random.default_rng(1)
    xs = set(int(v) for v in rng.integers(0, 2**63, 20000, dtype=np.uint64)) | set(range(4096))
    assert len({oracle.mix(x) for x in xs}) == len(xs)


@pytest.mark.parametrize("name", sorted(RECIPES))
def test_golden_block_and_tensor_digests(oracle, name):
    want_d, want_t = GOLD[name]
    T, bd = oracle.tensor_digest(RECIPES[name])
    assert [int(v) for v in bd] == want_d
    assert T == want_t


def test_zero_block_closed_form_from_generator(oracle):
    # word i of a zero block contributes mix(i*G) = i-th generator output (i >= 1); mix(0) = 0
    acc = 0
    for v in splitmix64_stream(0, 511):
        acc ^= v
    assert oracle.block_digest(np.zeros(4096, np.uint8)) == acc == GOLD["zeros_4096"][0][0]


def test_pad_suffix_closed_form(oracle):
    stream = [0] + splitmix64_stream(0, 511)  # stream[i] = mix(i*G)
    want = GOLD["pad_suffix"][0]
    for k, w in zip((0, 1, 256, 511, 512), want):
        acc = 0
        for i in range(k, 512):
            acc ^= stream[i]
        assert acc == w
        # words below k cancel their constants (mix(0) = 0); words from k on are absent (zero)
        assert oracle.block_digest(words_le(i * G for i in range(k))) == w


def test_every_word_position_and_byte_order(oracle):
    # Block whose word j is j*G ^ k*G and every other word i is i*G: all terms vanish
    # except mix(k*G), a textbook output.  Wrong index base, wrong word stride, wrong
    # endianness or a dropped word breaks it.
    stream = [0] + splitmix64_stream(0, 600)
    base = [(i * G) & M64 for i in range(512)]
    for j in range(512):
        k = (j * 7 + 5) % 600 + 1
        w = list(base)
        w[j] ^= (k * G) & M64
        raw = b"".join(int(v).to_bytes(8, "little") for v in w)
        assert oracle.block_digest(raw) == stream[k], j


def test_partial_word_tail_is_little_endian_zero_filled(oracle):
    rng = np.random.default_rng(7)
    for m in (1, 2, 3, 7, 8, 9, 15, 16, 17, 4087, 4095):
        x = rng.integers(0, 256, m, dtype=np.uint8)
        padded = np.zeros(4096, np.uint8)
        padded[:m] = x
        assert oracle.block_digest(x) == oracle.block_digest(padded)
    # the single byte b at offset 8*j + s is the word (b << 8s) at index j
    stream = [0] + splitmix64_stream(0, 511)
    zero = GOLD["zeros_4096"][0][0]
    for j, s in ((0, 0), (5, 3), (511, 7)):
        # against the zero block only term j changes: mix(j*G) is replaced by mix(w ^ j*G)
        x = np.zeros(8 * j + s + 1, np.uint8)
        x[-1] = 0xA5
        w = 0xA5 << (8 * s)
        want = zero ^ stream[j] ^ oracle.mix(w ^ ((j * G) & M64))
        assert oracle.block_digest(x) == want


def test_tensor_digest_block_index_is_bound_in(oracle):
    rng = np.random.default_rng(11)
    a = rng.integers(0, 256, 4096, dtype=np.uint8)
    b = rng.integers(0, 256, 4096, dtype=np.uint8)
    Tab, dab = oracle.tensor_digest(np.concatenate([a, b]))
    Tba, dba = oracle.tensor_digest(np.concatenate([b, a]))
    assert list(dab) == list(dba)[::-1]  # block digests do not depend on the position
    assert Tab != Tba  # the tensor digest does
    Ta, da = oracle.tensor_digest(a)
    assert Ta != int(da[0])  # block 0 is mixed, not passed through
    assert oracle.tensor_digest(np.zeros(0, np.uint8))[0] == 0
    # T of one block whose digest is 0 is mix(0) = 0 (block index 0 contributes 0*G)
    assert oracle.tensor_digest(RECIPES["words_iG_512"])[0] == 0
    # same block at index 1 contributes mix(1*G) = first generator output
    two = np.concatenate([RECIPES["words_iG_512"], RECIPES["words_iG_512"]])
    assert oracle.tensor_digest(two)[0] == splitmix64_stream(0, 1)[0]
    # ... and at indices 1..5 the XOR of outputs 1..5
    six = np.concatenate([RECIPES["words_iG_512"]] * 6)
    acc = 0
    for v in splitmix64_stream(0, 5):
        acc ^= v
    assert oracle.tensor_digest(six)[0] == acc


def test_zero_padding_versus_length(oracle):
    rng = np.random.default_rng(3)
    x = rng.integers(0, 256, 5000, dtype=np.uint8)
    T0, d0 = oracle.tensor_digest(x)
    T1, d1 = oracle.tensor_digest(np.concatenate([x, np.zeros(8192 - 5000, np.uint8)]))
    assert T0 == T1 and list(d0) == list(d1)  # same block count, zero fill: same digest
    T2, d2 = oracle.tensor_digest(np.concatenate([x, np.zeros(8192 - 5000 + 1, np.uint8)]))
    assert T2 != T0 and len(d2) == 3  # one more (all-zero) block changes T


def test_every_single_bit_flip_is_detected_and_localised(oracle):
    rng = np.random.default_rng(5)
    L = 4096 + 4096 + 24
    x = rng.integers(0, 256, L, dtype=np.uint8)
    rec = oracle.make_record([(42, 0, 0, L)])
    T0, d0 = oracle.tensor_digest(x)
    seen_T = {T0}
    for byte in list(range(0, 64)) + list(range(4090, 4102)) + list(range(L - 24, L)) + [2000, 6000]:
        for bit in range(8):
            y = x.copy()
            y[byte] ^= 1 << bit
            T1, d1 = oracle.tensor_digest(y)
            assert T1 != T0
            seen_T.add(T1)
            n, mm = oracle.verify(rec, d1, d0, cap=8)
            assert n == 1 and int(mm[0]["tensor_id"]) == 42 and int(mm[0]["block"]) == byte // 4096
    assert len(seen_T) > 8 * 100  # all distinct


def test_single_bit_flip_exhaustive_on_one_block(oracle):
    rng = np.random.default_rng(6)
    x = rng.integers(0, 256, 520, dtype=np.uint8)  # 65 words; every bit of it
    D0 = oracle.block_digest(x)
    digests = set()
    for byte in range(520):
        for bit in range(8):
            y = x.copy()
            y[byte] ^= 1 << bit
            digests.add(oracle.block_digest(y))
    assert D0 not in digests and len(digests) == 520 * 8


def _random_record(rng, n, max_bytes, guard=64):
    sizes = [int(rng.integers(0, max_bytes + 1)) for _ in range(n)]
    src, off = [], 0
    for s in sizes:
        src.append(off)
        off += (s + 15) // 16 * 16
    image_bytes = off
    order = rng.permutation(n)
    dst, off = [0] * n, guard
    for t in order:
        dst[t] = off
        off += (sizes[t] + 15) // 16 * 16 + guard
    rows = [(1000 + 3 * t, src[t], dst[t], sizes[t]) for t in range(n)]
    return rows, image_bytes, off


def test_restore_copies_exactly_and_digests_what_it_copied(oracle):
    rng = np.random.default_rng(21)
    rows, image_bytes, slab_bytes = _random_record(rng, 40, 20000)
    rec = oracle.make_record(rows)
    image = rng.integers(0, 256, image_bytes, dtype=np.uint8)
    slab = np.full(slab_bytes, 0xEE, np.uint8)
    rc, bd, td = oracle.restore(rec, image, slab)
    assert rc == 0
    touched = np.zeros(slab_bytes, bool)
    base, total = oracle.block_bases(rec)
    assert total == sum((r[3] + 4095) // 4096 for r in rows) == bd.size
    for t, (tid, so, do, nb) in enumerate(rows):
        assert np.array_equal(slab[do : do + nb], image[so : so + nb])  # brute-force byte compare
        touched[do : do + nb] = True
        T, d = oracle.tensor_digest(image[so : so + nb])  # digest of the image segment
        assert T == int(td[t]) and list(d) == list(bd[int(base[t]) : int(base[t]) + len(d)])
    assert np.all(slab[~touched] == 0xEE)  # nothing outside [dst, dst+nbytes) was written
    rc2, bd2, td2 = oracle.digest(rec, slab)
    assert rc2 == 0 and np.array_equal(bd, bd2) and np.array_equal(td, td2)


def test_results_do_not_depend_on_record_order(oracle):
    rng = np.random.default_rng(22)
    rows, image_bytes, slab_bytes = _random_record(rng, 30, 9000)
    image = rng.integers(0, 256, image_bytes, dtype=np.uint8)
    slab_a, slab_b = np.zeros(slab_bytes, np.uint8), np.zeros(slab_bytes, np.uint8)
    rec_a = oracle.make_record(rows)
    perm = rng.permutation(len(rows))
    rec_b = oracle.make_record([rows[i] for i in perm])
    _, bd_a, td_a = oracle.restore(rec_a, image, slab_a)
    _, bd_b, td_b = oracle.restore(rec_b, image, slab_b)
    assert np.array_equal(slab_a, slab_b)
    base_a, _ = oracle.block_bases(rec_a)
    base_b, _ = oracle.block_bases(rec_b)
    for pos_b, t in enumerate(perm):
        assert td_b[pos_b] == td_a[t]
        nb = (rows[t][3] + 4095) // 4096
        assert np.array_equal(bd_b[int(base_b[pos_b]) : int(base_b[pos_b]) + nb], bd_a[int(base_a[t]) : int(base_a[t]) + nb])


def test_verify_agrees_with_byte_comparison(oracle):
    rng = np.random.default_rng(23)
    for trial in range(20):
        rows, image_bytes, slab_bytes = _random_record(rng, 12, 10000)
        rec = oracle.make_record(rows)
        image = rng.integers(0, 256, image_bytes, dtype=np.uint8)
        slab = np.zeros(slab_bytes, np.uint8)
        _, expected, _ = oracle.restore(rec, image, slab)
        # corrupt a few random bytes (possibly none)
        for _ in range(int(rng.integers(0, 4))):
            t = int(rng.integers(0, len(rows)))
            if rows[t][3] == 0:
                continue
            slab[rows[t][2] + int(rng.integers(0, rows[t][3]))] ^= 1 << int(rng.integers(0, 8))
        _, computed, _ = oracle.digest(rec, slab)
        want = []
        for tid, so, do, nb in rows:
            for b in range((nb + 4095) // 4096):
                lo, hi = b * 4096, min(nb, b * 4096 + 4096)
                if not np.array_equal(slab[do + lo : do + hi], image[so + lo : so + hi]):
                    want.append((tid, b))
        n, mm = oracle.verify(rec, computed, expected, cap=64)
        assert n == len(want) and [(int(m["tensor_id"]), int(m["block"])) for m in mm] == want
        n2, mm2 = oracle.verify(rec, computed, expected, cap=1)
        assert n2 == len(want) and len(mm2) == min(1, len(want))


def test_validation_status_codes(oracle):
    mk = oracle.make_record
    assert oracle.validate(mk([(1, 0, 0, 100), (2, 112, 112, 100)]), 1000, 1000) == oracle.OK
    assert oracle.validate(mk([(1, 8, 0, 100)]), 1000, 1000) == oracle.ERR_ALIGN
    assert oracle.validate(mk([(1, 0, 8, 100)]), 1000, 1000) == oracle.ERR_ALIGN
    assert oracle.validate(mk([(1, 992, 0, 16)]), 1000, 1000) == oracle.ERR_RANGE
    assert oracle.validate(mk([(1, 0, 0, 2**64 - 1)]), 1000, 1000) == oracle.ERR_RANGE
    assert oracle.validate(mk([(1, 0, 0, 100), (2, 112, 96, 100)]), 1000, 1000) == oracle.ERR_OVERLAP
    assert oracle.validate(mk([(1, 0, 0, 100), (1, 112, 112, 100)]), 1000, 1000) == oracle.ERR_DUP_ID
    # overlapping sources are legal; zero-length tensors overlap nothing
    assert oracle.validate(mk([(1, 0, 0, 100), (2, 0, 112, 100), (3, 0, 0, 0)]), 1000, 1000) == oracle.OK


def test_kv_restore_reduces_to_restore_and_tensor_digest(oracle):
    rng = np.random.default_rng(31)
    n_planes, n_blocks, bb, n_sel = 6, 11, 8192, 5
    k = bb // 4096
    plane_stride, block_stride = n_blocks * bb + 4096, bb
    pool = rng.integers(0, 256, n_planes * plane_stride, dtype=np.uint8)
    before = pool.copy()
    image = rng.integers(0, 256, n_planes * n_sel * bb, dtype=np.uint8)
    ips, iss = n_sel * bb, bb
    ids = np.array([7, -1, 0, 11, 10], np.int32)  # -1 and 11 are out of range
    rc, bd, kd, skipped = oracle.kv_restore(pool, plane_stride, block_stride, n_planes, n_blocks, bb, image, ips, iss, ids)
    assert rc == 0 and skipped == 2
    want_pool = before.copy()
    for j, blk in enumerate(ids):
        ok = 0 <= blk < n_blocks
        cat = []
        for p in range(n_planes):
            seg = image[p * ips + j * iss : p * ips + j * iss + bb]
            if ok:
                want_pool[p * plane_stride + blk * block_stride :][:bb] = seg
            cat.append(seg)
            for c in range(k):
                got = int(bd[(j * n_planes + p) * k + c])
                assert got == (oracle.block_digest(seg[c * 4096 : (c + 1) * 4096]) if ok else 0)
        T, _ = oracle.tensor_digest(np.concatenate(cat))
        assert int(kd[j]) == (T if ok else 0)
    assert np.array_equal(pool, want_pool)


def test_capture_is_the_inverse_of_restore(oracle):
    rng = np.random.default_rng(51)
    rows, image_bytes, slab_bytes = _random_record(rng, 35, 15000)
    rec = oracle.make_record(rows)
    slab = rng.integers(0, 256, slab_bytes, dtype=np.uint8)
    image = np.full(image_bytes, 0xC3, np.uint8)
    rc, bd, td = oracle.capture(rec, image, slab)
    assert rc == 0
    covered = np.zeros(image_bytes, bool)
    for tid, so, do, nb in rows:
        assert np.array_equal(image[so : so + nb], slab[do : do + nb])  # brute-force byte compare
        covered[so : so + nb] = True
    assert np.all(image[~covered] == 0xC3)  # image bytes no entry covers are left alone
    # the digests of a capture are the digests of the destinations where they lie ...
    rc2, bd2, td2 = oracle.digest(rec, slab)
    assert np.array_equal(bd, bd2) and np.array_equal(td, td2)
    # ... and restoring the captured image gives back the same bytes and the same digests
    slab2 = np.zeros(slab_bytes, np.uint8)
    rc3, bd3, td3 = oracle.restore(rec, image, slab2)
    assert rc3 == 0 and np.array_equal(bd3, bd) and np.array_equal(td3, td)
    for tid, so, do, nb in rows:
        assert np.array_equal(slab2[do : do + nb], slab[do : do + nb])
    # two tensors packed onto the same image bytes are refused by capture (restore accepts shared sources)
    shared = oracle.make_record([(1, 0, 0, 100), (2, 0, 112, 100)])
    assert oracle.validate(shared, 1000, 1000) == oracle.OK
    assert oracle.capture(shared, np.zeros(1000, np.uint8), np.zeros(1000, np.uint8))[0] == oracle.ERR_OVERLAP


def test_kv_capture_is_the_inverse_of_kv_restore(oracle):
    rng = np.random.default_rng(52)
    n_planes, n_blocks, bb = 5, 13, 8192
    ids = np.array([3, 12, -2, 0, 13, 7], np.int32)  # -2 and 13 are out of range
    plane_stride, ips = n_blocks * bb + 512, len(ids) * bb
    pool = rng.integers(0, 256, n_planes * plane_stride, dtype=np.uint8)
    image = np.full(n_planes * ips, 0x77, np.uint8)
    rc, bd, kd, skipped = oracle.kv_capture(pool, plane_stride, bb, n_planes, n_blocks, bb, image, ips, bb, ids)
    assert rc == 0 and skipped == 2
    for j, blk in enumerate(ids):
        for p in range(n_planes):
            slot = image[p * ips + j * bb :][:bb]
            if 0 <= blk < n_blocks:
                assert np.array_equal(slot, pool[p * plane_stride + blk * bb :][:bb])
            else:
                assert np.all(slot == 0x77)
    # scattering the captured image back reproduces the pool and the same digests
    pool2 = pool.copy()
    for j, blk in enumerate(ids):
        if 0 <= blk < n_blocks:
            for p in range(n_planes):
                pool2[p * plane_stride + blk * bb :][:bb] = 0
    rc2, bd2, kd2, skipped2 = oracle.kv_restore(pool2, plane_stride, bb, n_planes, n_blocks, bb, image, ips, bb, ids)
    assert rc2 == 0 and skipped2 == 2 and np.array_equal(pool2, pool)
    assert np.array_equal(bd2, bd) and np.array_equal(kd2, kd)


def test_kv_digest_is_the_tensor_digest_of_the_block_planes_in_place(oracle):
    rng = np.random.default_rng(53)
    n_planes, n_blocks, bb = 4, 9, 12288
    k = bb // 4096
    ids = np.array([8, 0, 9, 4, -1], np.int32)  # 9 and -1 are out of range
    plane_stride, block_stride = n_blocks * bb + 1024, bb
    pool = rng.integers(0, 256, n_planes * plane_stride, dtype=np.uint8)
    before = pool.copy()
    rc, bd, kd, skipped = oracle.kv_digest(pool, plane_stride, block_stride, n_planes, n_blocks, bb, ids)
    assert rc == 0 and skipped == 2
    assert np.array_equal(pool, before)  # read-only
    for j, blk in enumerate(ids):
        ok = 0 <= blk < n_blocks
        planes = [before[p * plane_stride + blk * block_stride :][:bb] for p in range(n_planes)] if ok else []
        for p in range(n_planes):
            for c in range(k):
                want = oracle.block_digest(planes[p][c * 4096 : (c + 1) * 4096]) if ok else 0
                assert int(bd[(j * n_planes + p) * k + c]) == want
        assert int(kd[j]) == (oracle.tensor_digest(np.concatenate(planes))[0] if ok else 0)
    # it is what a capture of the same blocks reports, and what restoring that capture reports
    image = np.zeros(n_planes * len(ids) * bb, np.uint8)
    rc, bd2, kd2, _ = oracle.kv_capture(before, plane_stride, block_stride, n_planes, n_blocks, bb, image, len(ids) * bb, bb, ids)
    assert rc == 0 and np.array_equal(bd2, bd) and np.array_equal(kd2, kd)
    # one flipped bit in one plane of block 4 changes exactly that 4 KiB block's digest and that slot's KV digest
    pool[2 * plane_stride + 4 * block_stride + 5000] ^= 0x20
    rc, bd3, kd3, _ = oracle.kv_digest(pool, plane_stride, block_stride, n_planes, n_blocks, bb, ids)
    diff = np.nonzero(bd3 != bd)[0]
    assert diff.tolist() == [(3 * n_planes + 2) * k + 1]
    assert np.nonzero(kd3 != kd)[0].tolist() == [3]


def test_kv_verify_agrees_with_byte_comparison_of_pool_blocks_and_image_slots(oracle):
    """The pin of kv_verify: put an image into a pool, damage pool bytes by hand, and compare what kv_verify names
    (from the digests of the damaged pool against the digests the restore reported) with a brute-force byte
    comparison of every pool block against its image slot, 4 KiB at a time, walked in list order."""
    rng = np.random.default_rng(54)
    n_planes, n_blocks, bb = 3, 11, 12288
    k = bb // 4096
    ids = np.array([7, -3, 2, 10, 11, 0, 5], np.int32)  # -3 and 11 are out of range
    plane_stride, ips = n_blocks * bb + 256, len(ids) * bb
    pool = rng.integers(0, 256, n_planes * plane_stride, dtype=np.uint8)
    image = rng.integers(0, 256, n_planes * ips, dtype=np.uint8)
    rc, expected, _, skipped = oracle.kv_restore(pool, plane_stride, bb, n_planes, n_blocks, bb, image, ips, bb, ids)
    assert rc == 0 and skipped == 2
    rc, computed, _, _ = oracle.kv_digest(pool, plane_stride, bb, n_planes, n_blocks, bb, ids)
    assert oracle.kv_verify(n_planes, n_blocks, bb, ids, computed, expected, 8)[0] == 0
    # host-made damage: single bits in chosen (block id, plane, sub-block), plus one in a block that is not in the list
    damage = [(2, 0, 1), (7, 2, 2), (7, 0, 0), (0, 1, 0), (5, 2, 2), (5, 2, 0)]
    for blk, p, c in damage:
        pool[p * plane_stride + blk * bb + c * 4096 + int(rng.integers(0, 4096))] ^= 1 << int(rng.integers(0, 8))
    pool[1 * plane_stride + 3 * bb + 17] ^= 0xFF  # block 3 is not selected: must not show up
    rc, computed, _, _ = oracle.kv_digest(pool, plane_stride, bb, n_planes, n_blocks, bb, ids)

    def brute():
        out = []
        for j, blk in enumerate(ids):
            if not 0 <= blk < n_blocks:
                continue
            for p in range(n_planes):
                for c in range(k):
                    a = pool[p * plane_stride + blk * bb + c * 4096 :][:4096]
                    b = image[p * ips + j * bb + c * 4096 :][:4096]
                    if not np.array_equal(a, b):
                        out.append((int(blk), p, c, j))
        return out

    want = brute()
    assert sorted((b, p, c) for b, p, c, _ in want) == sorted(damage)
    count, recs = oracle.kv_verify(n_planes, n_blocks, bb, ids, computed, expected, 16)
    assert count == len(want) == 6
    assert [(int(r["block_id"]), int(r["plane"]), int(r["sub_block"]), int(r["list_pos"])) for r in recs] == want
    # cap below the count: the total is still reported, the list is cut, its order unchanged
    count, recs = oracle.kv_verify(n_planes, n_blocks, bb, ids, computed, expected, 4)
    assert count == 6 and [(int(r["block_id"]), int(r["plane"]), int(r["sub_block"]), int(r["list_pos"])) for r in recs] == want[:4]
    assert oracle.kv_verify(n_planes, n_blocks, bb, ids, computed, expected, 0)[0] == 6
    # slots of skipped ids are never reported, whatever they hold
    noisy = computed.copy()
    noisy[(1 * n_planes + 0) * k + 0] ^= 1   # list position 1 is id -3
    noisy[(4 * n_planes + 2) * k + 2] ^= 1   # list position 4 is id 11
    assert oracle.kv_verify(n_planes, n_blocks, bb, ids, noisy, expected, 16)[0] == 6


def test_oracle_has_not_drifted_from_its_stored_outputs(oracle):
    """tests/golden/oracle_regression.txt was written by tests/golden/make_oracle_regression.py, which calls only the
    oracle: a drift alarm (any later change to the oracle's arithmetic must be deliberate), not a correctness pin."""
    import importlib.util
    import os

    here = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
    spec = importlib.util.spec_from_file_location("make_oracle_regression", os.path.join(here, "make_oracle_regression.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    with open(os.path.join(here, "oracle_regression.txt")) as f:
        assert f.read() == mod.render()
