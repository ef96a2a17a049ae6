/*
 * gms_oracle.c -- plain, slow, single-threaded CPU statement of what the
 * restore / digest / verify / kv-restore path computes.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT PRODUCT CODE.  Only the test-suite, the
 * smoke check and the benchmark's CPU-baseline leg may call it.  It shares no
 * code, header, table or constant generator with the CUDA library and must
 * never be reached from the product path.
 *
 * What it states.  The paper (Section 3.2, GMS; Section 3.3, Snapshots with
 * GMS; Section 4, GMS paragraph) describes model state that lives in
 * service-owned device allocations, a writer that notes every tensor's place
 * before it commits, a cold-service path in which a fresh writer fills those
 * allocations again, and a warm path in which a replacement engine reuses the
 * surviving bytes provided they are still intact (Section 2.2).  The paper
 * gives no digest and no record format; the library fixes both, and this file
 * writes that definition out literally:
 *
 *   mix(z)   : the three xor-shift / multiply stages of the SplitMix64 output
 *              function, without the generator's additive state step.
 *   D(block) : a block is at most 4096 bytes, zero-extended to 4096; with w_i
 *              the little-endian 64-bit word at byte 8i (i = 0..511),
 *              D = XOR_i mix(w_i ^ (i * G)),   G = 0x9E3779B97F4A7C15.
 *   T(tensor): blocks are cut relative to the tensor's first byte;
 *              T = XOR_b mix(D_b ^ (b * G)); a tensor of 0 bytes has T = 0.
 *
 * All arithmetic is on uint64_t and wraps mod 2^64.  No blocking, no tables,
 * no algebraic shortcuts: one word at a time, in index order.
 *
 * Every function here is pinned by tests/test_oracle_pins.py against values
 * and properties that do not come from this file (published SplitMix64
 * outputs, closed forms, exhaustive bit flips, brute-force byte comparison).
 */
#include <stddef.h>
#include <stdint.h>
#include <string.h>

#define GMSO_BLOCK 4096u
#define GMSO_WORDS 512u
#define GMSO_G 0x9E3779B97F4A7C15ULL

/* status values returned by the validating entry points */
#define GMSO_OK 0
#define GMSO_ERR_NULL (-1)
#define GMSO_ERR_ALIGN (-2)
#define GMSO_ERR_RANGE (-3)
#define GMSO_ERR_OVERLAP (-4)
#define GMSO_ERR_DUP_ID (-5)

typedef struct {
    uint64_t tensor_id;  /* caller's name for the tensor                    */
    uint64_t src_offset; /* byte offset of the tensor in the packed image   */
    uint64_t dst_offset; /* byte offset of the destination inside dst_base  */
    uint64_t nbytes;     /* length in bytes (may be 0)                      */
} gmso_entry;

typedef struct {
    uint64_t tensor_id;
    uint64_t block; /* block index relative to the tensor */
} gmso_mismatch;

/* mix: SplitMix64 output function without the "+= G" state step. */
uint64_t gmso_mix(uint64_t z)
{
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}

/* D: digest of one block of m bytes, 0 <= m <= 4096, zero-extended. */
uint64_t gmso_block_digest(const uint8_t *x, size_t m)
{
    uint8_t padded[GMSO_BLOCK];
    uint64_t d = 0;
    memset(padded, 0, sizeof padded);
    if (m > GMSO_BLOCK) m = GMSO_BLOCK;
    if (m) memcpy(padded, x, m);
    for (uint64_t i = 0; i < GMSO_WORDS; ++i) {
        uint64_t w = 0;
        for (int k = 7; k >= 0; --k) w = (w << 8) | padded[8 * i + (uint64_t)k]; /* little endian */
        d ^= gmso_mix(w ^ (i * GMSO_G));
    }
    return d;
}

/* number of 4 KiB blocks a tensor of L bytes is cut into */
uint64_t gmso_num_blocks(uint64_t L) { return (L + GMSO_BLOCK - 1) / GMSO_BLOCK; }

/* T: digest of a tensor of L bytes; block digests optionally written out. */
uint64_t gmso_tensor_digest(const uint8_t *x, uint64_t L, uint64_t *block_digests)
{
    uint64_t nb = gmso_num_blocks(L), t = 0;
    for (uint64_t b = 0; b < nb; ++b) {
        uint64_t lo = b * GMSO_BLOCK;
        uint64_t hi = lo + GMSO_BLOCK < L ? lo + GMSO_BLOCK : L;
        uint64_t d = gmso_block_digest(x + lo, (size_t)(hi - lo));
        if (block_digests) block_digests[b] = d;
        t ^= gmso_mix(d ^ (b * GMSO_G));
    }
    return t;
}

/*
 * Validation of a layout record: 16-byte aligned source offsets and
 * destinations, sources inside the image, destinations inside the slab,
 * pairwise disjoint destinations, distinct ids.  Quadratic on purpose.
 */
int gmso_validate(const gmso_entry *e, size_t n, uint64_t image_bytes, uint64_t dst_bytes)
{
    if (n && !e) return GMSO_ERR_NULL;
    for (size_t t = 0; t < n; ++t) {
        if ((e[t].src_offset & 15u) || (e[t].dst_offset & 15u)) return GMSO_ERR_ALIGN;
        if (e[t].src_offset > image_bytes || e[t].nbytes > image_bytes - e[t].src_offset) return GMSO_ERR_RANGE;
        if (e[t].dst_offset > dst_bytes || e[t].nbytes > dst_bytes - e[t].dst_offset) return GMSO_ERR_RANGE;
    }
    for (size_t a = 0; a < n; ++a)
        for (size_t b = a + 1; b < n; ++b) {
            if (e[a].tensor_id == e[b].tensor_id) return GMSO_ERR_DUP_ID;
            if (e[a].nbytes && e[b].nbytes && e[a].dst_offset < e[b].dst_offset + e[b].nbytes &&
                e[b].dst_offset < e[a].dst_offset + e[a].nbytes)
                return GMSO_ERR_OVERLAP;
        }
    return GMSO_OK;
}

/* total number of digest blocks of a record, and each tensor's first block */
uint64_t gmso_block_bases(const gmso_entry *e, size_t n, uint64_t *base /* n entries, may be NULL */)
{
    uint64_t acc = 0;
    for (size_t t = 0; t < n; ++t) {
        if (base) base[t] = acc;
        acc += gmso_num_blocks(e[t].nbytes);
    }
    return acc;
}

/*
 * Restore: for each entry in record order copy its bytes from the image to its
 * destination, and digest the copied bytes.  block_digests has one slot per
 * block in record order (tensor t starts at the prefix sum of the block counts
 * before it); tensor_digests has one slot per entry.  Either may be NULL.
 */
int gmso_restore(const gmso_entry *e, size_t n, const uint8_t *image, uint64_t image_bytes, uint8_t *dst_base,
                 uint64_t dst_bytes, uint64_t *block_digests, uint64_t *tensor_digests)
{
    int rc = gmso_validate(e, n, image_bytes, dst_bytes);
    uint64_t base = 0;
    if (rc) return rc;
    if (n && (!image || !dst_base)) return GMSO_ERR_NULL;
    for (size_t t = 0; t < n; ++t) {
        uint8_t *dst = dst_base + e[t].dst_offset;
        if (e[t].nbytes) memcpy(dst, image + e[t].src_offset, (size_t)e[t].nbytes);
        uint64_t T = gmso_tensor_digest(dst, e[t].nbytes, block_digests ? block_digests + base : NULL);
        if (tensor_digests) tensor_digests[t] = T;
        base += gmso_num_blocks(e[t].nbytes);
    }
    return GMSO_OK;
}

/*
 * Capture: the inverse of restore (Section 3.1, step 3: device state is staged into a host-side image before it
 * is serialised; Section 3.2: what is captured at commit is what later reuse is checked against).  For each entry
 * in record order the tensor's bytes are copied from its destination into the packed image at src_offset, and
 * digested.  Image ranges must be pairwise disjoint here (two tensors packed onto the same image bytes would
 * overwrite each other), which restore does not require.  Image bytes that no entry covers are left alone.
 */
int gmso_capture(const gmso_entry *e, size_t n, uint8_t *image, uint64_t image_bytes, const uint8_t *dst_base,
                 uint64_t dst_bytes, uint64_t *block_digests, uint64_t *tensor_digests)
{
    int rc = gmso_validate(e, n, image_bytes, dst_bytes);
    uint64_t base = 0;
    if (rc) return rc;
    if (n && (!image || !dst_base)) return GMSO_ERR_NULL;
    for (size_t a = 0; a < n; ++a)
        for (size_t b = a + 1; b < n; ++b)
            if (e[a].nbytes && e[b].nbytes && e[a].src_offset < e[b].src_offset + e[b].nbytes &&
                e[b].src_offset < e[a].src_offset + e[a].nbytes)
                return GMSO_ERR_OVERLAP;
    for (size_t t = 0; t < n; ++t) {
        const uint8_t *src = dst_base + e[t].dst_offset;
        if (e[t].nbytes) memcpy(image + e[t].src_offset, src, (size_t)e[t].nbytes);
        uint64_t T = gmso_tensor_digest(image + e[t].src_offset, e[t].nbytes, block_digests ? block_digests + base : NULL);
        if (tensor_digests) tensor_digests[t] = T;
        base += gmso_num_blocks(e[t].nbytes);
    }
    return GMSO_OK;
}

/* Digest the destinations where they lie; nothing is written to them. */
int gmso_digest(const gmso_entry *e, size_t n, const uint8_t *dst_base, uint64_t dst_bytes, uint64_t *block_digests,
                uint64_t *tensor_digests)
{
    uint64_t base = 0;
    if (n && (!e || !dst_base)) return GMSO_ERR_NULL;
    for (size_t t = 0; t < n; ++t) {
        if (e[t].dst_offset > dst_bytes || e[t].nbytes > dst_bytes - e[t].dst_offset) return GMSO_ERR_RANGE;
        uint64_t T = gmso_tensor_digest(dst_base + e[t].dst_offset, e[t].nbytes,
                                        block_digests ? block_digests + base : NULL);
        if (tensor_digests) tensor_digests[t] = T;
        base += gmso_num_blocks(e[t].nbytes);
    }
    return GMSO_OK;
}

/*
 * Verify: the set of (tensor id, block) whose computed digest differs from the
 * expected one, ascending by (record position, block).  Returns the size of
 * the whole set; only the first `cap` members are written.
 */
uint64_t gmso_verify(const gmso_entry *e, size_t n, const uint64_t *computed, const uint64_t *expected,
                     gmso_mismatch *out, uint64_t cap)
{
    uint64_t count = 0, base = 0;
    for (size_t t = 0; t < n; ++t) {
        uint64_t nb = gmso_num_blocks(e[t].nbytes);
        for (uint64_t b = 0; b < nb; ++b) {
            if (computed[base + b] != expected[base + b]) {
                if (count < cap) {
                    out[count].tensor_id = e[t].tensor_id;
                    out[count].block = b;
                }
                ++count;
            }
        }
        base += nb;
    }
    return count;
}

/*
 * Paged-KV subset restore (Section 6, "Preserving KV state": committed KV
 * blocks kept outside the engine and put back after recovery).  The pool is
 * n_planes planes (layer x {K,V}) of n_blocks blocks of block_bytes bytes.
 * Selected slot j of the packed image goes to pool block ids[j] in every
 * plane.  block_bytes is a multiple of 4096.  Digests:
 *   block_digests[(j * n_planes + p) * k + c]  for the c-th 4 KiB block of
 *       plane p of slot j, k = block_bytes / 4096;
 *   kv_digests[j] = XOR_q mix(D_q ^ q*G), q = p*k + c, i.e. the tensor digest
 *       of the slot's planes concatenated in plane order.
 * An id outside [0, n_blocks) is skipped: nothing is copied, its digests are
 * 0, and *skipped is incremented.
 */
int gmso_kv_restore(uint8_t *pool_base, uint64_t plane_stride, uint64_t block_stride, uint32_t n_planes,
                    uint32_t n_blocks, uint32_t block_bytes, const uint8_t *image, uint64_t img_plane_stride,
                    uint64_t img_slot_stride, const int32_t *ids, uint32_t n_sel, uint64_t *block_digests,
                    uint64_t *kv_digests, uint64_t *skipped)
{
    uint64_t k = block_bytes / GMSO_BLOCK, skip = 0;
    if (block_bytes == 0 || block_bytes % GMSO_BLOCK) return GMSO_ERR_ALIGN;
    if (n_sel && (!pool_base || !image || !ids)) return GMSO_ERR_NULL;
    for (uint32_t j = 0; j < n_sel; ++j) {
        int ok = ids[j] >= 0 && (uint32_t)ids[j] < n_blocks;
        uint64_t K = 0;
        if (!ok) ++skip;
        for (uint32_t p = 0; p < n_planes; ++p) {
            const uint8_t *src = image + (uint64_t)p * img_plane_stride + (uint64_t)j * img_slot_stride;
            uint8_t *dst = ok ? pool_base + (uint64_t)p * plane_stride + (uint64_t)ids[j] * block_stride : NULL;
            if (ok) memcpy(dst, src, block_bytes);
            for (uint64_t c = 0; c < k; ++c) {
                uint64_t q = (uint64_t)p * k + c;
                uint64_t d = ok ? gmso_block_digest(dst + c * GMSO_BLOCK, GMSO_BLOCK) : 0;
                if (block_digests) block_digests[((uint64_t)j * n_planes + p) * k + c] = d;
                if (ok) K ^= gmso_mix(d ^ (q * GMSO_G));
            }
        }
        if (kv_digests) kv_digests[j] = ok ? K : 0;
    }
    if (skipped) *skipped = skip;
    return GMSO_OK;
}

/*
 * Paged-KV subset capture: the gather direction of the same extension (committed KV blocks are kept outside the
 * engine, Section 6).  Selected pool block ids[j] of every plane is copied into slot j of the packed image; digests
 * are laid out exactly as in gmso_kv_restore.  An id outside [0, n_blocks) is skipped: its image slot is left
 * alone, its digests are 0, and *skipped is incremented.
 */
int gmso_kv_capture(const uint8_t *pool_base, uint64_t plane_stride, uint64_t block_stride, uint32_t n_planes,
                    uint32_t n_blocks, uint32_t block_bytes, uint8_t *image, uint64_t img_plane_stride,
                    uint64_t img_slot_stride, const int32_t *ids, uint32_t n_sel, uint64_t *block_digests,
                    uint64_t *kv_digests, uint64_t *skipped)
{
    uint64_t k = block_bytes / GMSO_BLOCK, skip = 0;
    if (block_bytes == 0 || block_bytes % GMSO_BLOCK) return GMSO_ERR_ALIGN;
    if (n_sel && (!pool_base || !image || !ids)) return GMSO_ERR_NULL;
    for (uint32_t j = 0; j < n_sel; ++j) {
        int ok = ids[j] >= 0 && (uint32_t)ids[j] < n_blocks;
        uint64_t K = 0;
        if (!ok) ++skip;
        for (uint32_t p = 0; p < n_planes; ++p) {
            uint8_t *dst = image + (uint64_t)p * img_plane_stride + (uint64_t)j * img_slot_stride;
            if (ok) memcpy(dst, pool_base + (uint64_t)p * plane_stride + (uint64_t)ids[j] * block_stride, block_bytes);
            for (uint64_t c = 0; c < k; ++c) {
                uint64_t q = (uint64_t)p * k + c;
                uint64_t d = ok ? gmso_block_digest(dst + c * GMSO_BLOCK, GMSO_BLOCK) : 0;
                if (block_digests) block_digests[((uint64_t)j * n_planes + p) * k + c] = d;
                if (ok) K ^= gmso_mix(d ^ (q * GMSO_G));
            }
        }
        if (kv_digests) kv_digests[j] = ok ? K : 0;
    }
    if (skipped) *skipped = skip;
    return GMSO_OK;
}

/*
 * Paged-KV subset digest in place: the check that decides whether KV blocks that outlived an engine may be reused
 * (Section 6, "Preserving KV state", read together with Section 2.2: surviving state is reused only if intact).
 * Pool block ids[j] of every plane is digested where it lies; nothing is written to the pool.  Digests are laid
 * out exactly as in gmso_kv_restore.  An id outside [0, n_blocks) is skipped: digests 0, *skipped incremented.
 */
int gmso_kv_digest(const uint8_t *pool_base, uint64_t plane_stride, uint64_t block_stride, uint32_t n_planes,
                   uint32_t n_blocks, uint32_t block_bytes, const int32_t *ids, uint32_t n_sel, uint64_t *block_digests,
                   uint64_t *kv_digests, uint64_t *skipped)
{
    uint64_t k = block_bytes / GMSO_BLOCK, skip = 0;
    if (block_bytes == 0 || block_bytes % GMSO_BLOCK) return GMSO_ERR_ALIGN;
    if (n_sel && (!pool_base || !ids)) return GMSO_ERR_NULL;
    for (uint32_t j = 0; j < n_sel; ++j) {
        int ok = ids[j] >= 0 && (uint32_t)ids[j] < n_blocks;
        uint64_t K = 0;
        if (!ok) ++skip;
        for (uint32_t p = 0; p < n_planes; ++p) {
            const uint8_t *blk = ok ? pool_base + (uint64_t)p * plane_stride + (uint64_t)ids[j] * block_stride : NULL;
            for (uint64_t c = 0; c < k; ++c) {
                uint64_t q = (uint64_t)p * k + c;
                uint64_t d = ok ? gmso_block_digest(blk + c * GMSO_BLOCK, GMSO_BLOCK) : 0;
                if (block_digests) block_digests[((uint64_t)j * n_planes + p) * k + c] = d;
                if (ok) K ^= gmso_mix(d ^ (q * GMSO_G));
            }
        }
        if (kv_digests) kv_digests[j] = ok ? K : 0;
    }
    if (skipped) *skipped = skip;
    return GMSO_OK;
}

/*
 * Paged-KV verify: the trust decision for KV state that outlived an engine (Section 6, "Preserving KV state",
 * read with the intact-state rule of Section 2.2), in terms a block manager can act on.  computed and expected
 * are digest arrays laid out as gmso_kv_restore / gmso_kv_digest lay them out, slot (j * n_planes + p) * k + c.
 * The result is the set of (pool block id, plane, 4 KiB sub-block) whose digests differ, in ascending
 * (list position j, plane p, sub-block c) order; an id outside [0, n_blocks) was never copied or digested and is
 * never reported, whatever its slots hold.  Returns the size of the whole set; only the first `cap` members are
 * written.
 */
typedef struct {
    uint32_t block_id;  /* ids[j]                                   */
    uint32_t plane;     /* p                                        */
    uint32_t sub_block; /* c: 4 KiB block inside the KV block       */
    uint32_t list_pos;  /* j: position of the block in the id list  */
} gmso_kv_mismatch;

uint64_t gmso_kv_verify(uint32_t n_planes, uint32_t n_blocks, uint32_t block_bytes, const int32_t *ids, uint32_t n_sel,
                        const uint64_t *computed, const uint64_t *expected, gmso_kv_mismatch *out, uint64_t cap)
{
    uint64_t k = block_bytes / GMSO_BLOCK, count = 0;
    for (uint32_t j = 0; j < n_sel; ++j) {
        if (ids[j] < 0 || (uint32_t)ids[j] >= n_blocks) continue;
        for (uint32_t p = 0; p < n_planes; ++p)
            for (uint64_t c = 0; c < k; ++c) {
                uint64_t slot = ((uint64_t)j * n_planes + p) * k + c;
                if (computed[slot] != expected[slot]) {
                    if (count < cap) {
                        out[count].block_id = (uint32_t)ids[j];
                        out[count].plane = p;
                        out[count].sub_block = (uint32_t)c;
                        out[count].list_pos = j;
                    }
                    ++count;
                }
            }
    }
    return count;
}
