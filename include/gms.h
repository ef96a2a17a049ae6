/*
 * gms.h -- C ABI of the restore / digest / verify data path of a GPU Memory
 * Service (GMS), written for NVIDIA B200 (sm_100a).
 *
 * Background (paper: "Fast Recovery for LLM Serving via Decoupled Device
 * Memory Lifetime in Dynamo").  Section 3.2 moves model state into device
 * allocations owned by a per-GPU service so that it outlives an engine:
 * a writer populates the allocations and commits them, later engines attach
 * read-only.  Section 4 (GMS paragraph) adds that the writer notes where each
 * tensor lies before it commits and that, when the service comes up cold, a
 * fresh writer fills the model state in again while the process is restored.
 * Section 3.1 models the cost of that as S / B_eff, and Section 5.2 observes
 * that the checkpoint tool in use moves device memory piece by piece, far
 * below what the link could carry.
 * Section 2.2 allows reuse of surviving allocations only if their contents are
 * intact.  The paper leaves the bulk data path and the integrity check
 * unspecified; this library is that path:
 *
 *   gms_manifest_build   the recorded tensor layout, turned into a work list
 *   gms_restore          scatter a packed snapshot image into the allocations,
 *                        digesting every 4 KiB block in the same pass
 *   gms_digest           digest surviving allocations in place (no writes)
 *   gms_verify           compare digests with the ones recorded at commit and
 *                        name the blocks that differ
 *   gms_kv_restore       scatter a subset of paged KV blocks (Section 6,
 *                        "Preserving KV state") through a block-index list
 *
 * The digest (fixed by this library, not by the paper; all arithmetic on
 * uint64_t, wrapping):
 *   mix(z):  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9;
 *            z = (z ^ (z >> 27)) * 0x94D049BB133111EB;  return z ^ (z >> 31);
 *   block digest  D   = XOR_{i<512} mix(w_i ^ i*G), G = 0x9E3779B97F4A7C15,
 *            w_i the little-endian u64 words of the block, a block shorter
 *            than 4096 bytes being extended with zero bytes;
 *   tensor digest T   = XOR_{b<nb} mix(D_b ^ b*G), blocks cut relative to the
 *            tensor's first byte, nb = ceil(nbytes / 4096); nbytes = 0: T = 0.
 * Results are exact integers; every output of this library is bit-reproducible.
 *
 * Conventions.
 *  - Every function returns int: GMS_OK (0) or a negative GMS_ERR_* value.
 *    Nothing throws, aborts or traps.  Host-detectable errors are returned
 *    before any device work is enqueued.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *    stream).  Device work is asynchronous with respect to the host; outputs
 *    are valid once the stream has been synchronised.
 *  - Pointers are marked (device), (host) or (device-accessible).  The caller
 *    owns every buffer it passes and keeps it alive until the stream work has
 *    completed.  The library allocates only the manifest's own small tables
 *    (by default 32 bytes per 16 KiB of payload -- 31 MB for a 16 GB manifest --
 *    plus 8 bytes per 4 KiB block once digests have been recorded, and a second
 *    copy of the 32-byte records, sorted by source offset, once gms_restore_fd
 *    or gms_restore_staged has been used on the manifest).
 *  - Calls that use the same manifest must not overlap on the GPU (they share
 *    the manifest's work counter and status word); enqueue them on one stream
 *    or order them with events.
 */
#ifndef GMS_H
#define GMS_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define GMS_BLOCK_BYTES 4096u

/* status codes */
#define GMS_OK 0
#define GMS_ERR_NULL (-1)     /* a required pointer is NULL                                   */
#define GMS_ERR_ALIGN (-2)    /* src_offset or dst not 16-byte aligned; bad block_bytes       */
#define GMS_ERR_RANGE (-3)    /* src_offset + nbytes exceeds the image, or overflows          */
#define GMS_ERR_OVERLAP (-4)  /* two destination ranges intersect                             */
#define GMS_ERR_DUP_ID (-5)   /* two entries carry the same tensor_id                         */
#define GMS_ERR_NOMEM (-6)    /* host or device allocation of the manifest's tables failed    */
#define GMS_ERR_CUDA (-7)     /* a CUDA runtime call failed; text via gms_last_cuda_error()   */
#define GMS_ERR_KIND (-8)     /* image_kind is not one of GMS_SRC_*                           */
#define GMS_ERR_TIMEOUT (-9)  /* a bounded device-side wait gave up (see device status word)  */
#define GMS_ERR_STATE (-10)   /* manifest has no device tables / no recorded digests          */
#define GMS_ERR_ARG (-11)     /* an argument is out of its documented range                   */
#define GMS_ERR_TOO_LARGE (-12) /* more digest blocks than gms_verify_flat_noalloc has room for */
#define GMS_ERR_IO (-13)      /* a file read failed or the file is shorter than the image     */

/* where the packed snapshot image lives */
#define GMS_SRC_DEVICE 0u      /* device memory (a staging buffer in HBM)                     */
#define GMS_SRC_HOST_MAPPED 1u /* pinned host memory mapped into the device address space     */

/* gms_manifest_build flags */
#define GMS_BUILD_HOST_ONLY 1u /* validate and build the work list on the host only (no CUDA
                                  call is made; device entry points return GMS_ERR_STATE)     */
#define GMS_BUILD_SELFTEST_STALL 2u /* self-test of the bounded waits, for test suites only: in every
                                  gms_restore / gms_capture / gms_digest of this manifest the barrier of
                                  the first block of chunk 0 is told to expect 16 bytes that are never
                                  sent, so the warp that claims it gives up after its wait limit (2 s),
                                  sets GMS_DEV_TIMEOUT, waits at most one more limit (2 s in all, not
                                  per copy) for the copies it still has in flight, and returns: the call
                                  ends by itself about 4 s after it began; the other warps finish their
                                  work.  Nothing faults; outputs of that call are incomplete by design. */

/* bits of the device status word */
#define GMS_DEV_TIMEOUT 1ull   /* a warp gave up waiting for one of its own bulk copies (2 s), then
                                  spent up to 2 s more draining the rest: worst case 4 s per call  */

typedef struct gms_manifest gms_manifest; /* opaque */

/* One recorded tensor layout (Section 4: what the writing client notes for each tensor before it commits). */
typedef struct {
    uint64_t tensor_id;  /* caller's identifier, unique within a manifest                     */
    uint64_t src_offset; /* byte offset of the tensor in the packed image, 16-byte aligned    */
    void *dst;           /* (device) destination, 16-byte aligned                             */
    uint64_t nbytes;     /* length in bytes, any value >= 0                                   */
} gms_entry;

typedef struct {
    uint64_t tensor_id; /* as given in the entry                                              */
    uint64_t block;     /* 4 KiB block index relative to the tensor's first byte              */
} gms_mismatch;

/*
 * gms_manifest_build -- Section 4, GMS paragraph (layout record made before
 * commit); Section 3.2 (the allocations it describes).
 * Validates `entries` (host, n of them) against an image of `image_bytes`
 * bytes and builds the work list that gms_restore / gms_digest walk: every
 * tensor is cut into chunks of 4 blocks (16 KiB; fewer for manifests too small
 * to give every warp two chunks, never more than 32) so that thousands of small
 * and a few huge tensors are served by one persistent launch.
 * Block digests are laid out in entry order: tensor t owns slots
 * [first_block(t), first_block(t) + ceil(nbytes_t/4096)).
 * The host's part is proportional to the number of tensors (validation, per-tensor
 * positions); the chunk records themselves are written by a kernel on the device,
 * on a stream of the library's own, and the call returns when they are complete
 * (it does not wait for work the caller has queued on other streams).
 * Errors: NULL, ALIGN, RANGE, OVERLAP (destinations; overlapping sources are
 * legal), DUP_ID, NOMEM, CUDA.  nbytes == 0 is legal (no blocks, T = 0).
 * Bytes of a destination beyond nbytes are never written.
 * On success *out owns host and (unless GMS_BUILD_HOST_ONLY) device tables on
 * the current device; release it with gms_manifest_destroy.
 */
int gms_manifest_build(const gms_entry *entries, size_t n, uint64_t image_bytes, uint32_t flags, gms_manifest **out);
int gms_manifest_destroy(gms_manifest *m);

/* Sizes of the outputs: number of entries, of digest blocks, and of payload bytes. */
int gms_manifest_info(const gms_manifest *m, uint64_t *n_tensors, uint64_t *n_blocks, uint64_t *payload_bytes);
/* First digest-block slot of entry `entry_index`. */
int gms_manifest_block_base(const gms_manifest *m, size_t entry_index, uint64_t *first_block);
/* Work-list introspection (host): number of chunks, and chunk `i` as
 * (entry index, byte offset inside the tensor, bytes).  Chunks partition every tensor. */
int gms_manifest_chunk_count(const gms_manifest *m, uint64_t *n_chunks);
int gms_manifest_chunk(const gms_manifest *m, uint64_t i, uint64_t *entry_index, uint64_t *tensor_byte_offset,
                       uint64_t *nbytes);

/*
 * gms_manifest_set_expected -- Section 3.2: commit makes the model state
 * immutable; the digests recorded at that moment are what later reuse is
 * checked against.  Copies n_blocks block digests (device) into the manifest
 * (device-to-device, on `stream`).
 */
int gms_manifest_set_expected(gms_manifest *m, const uint64_t *d_block_digests, void *stream);

/*
 * gms_restore -- Section 4 (cold-service repopulation), Section 3.3
 * (reconstruction after a device-invalidating failure), cost model S/B_eff of
 * Section 3.1.  For every entry: dst[0, nbytes) <- image[src_offset, +nbytes),
 * and, in the same pass over the bytes, D for each block and T for each tensor.
 *   image            (device-accessible) start of the packed image:
 *                    device memory for GMS_SRC_DEVICE, the device-side
 *                    address of pinned mapped host memory for
 *                    GMS_SRC_HOST_MAPPED; 16-byte aligned
 *   d_block_digests  (device) n_blocks u64, may be NULL
 *   d_tensor_digests (device) n u64, may be NULL
 * One persistent kernel (plus a one-block prologue that clears accumulators);
 * no per-tensor launches.  Errors: NULL, ALIGN, KIND, STATE, CUDA.
 */
int gms_restore(const gms_manifest *m, const void *image, uint32_t image_kind, uint64_t *d_block_digests,
                uint64_t *d_tensor_digests, void *stream);

/*
 * gms_capture -- the inverse of gms_restore: Section 3.1, step 3 (device state is staged into a
 * host-side image before it is serialised) and Section 3.2 (what is recorded at commit is what
 * later reuse is checked against).  For every entry: image[src_offset, +nbytes) <- dst[0, nbytes),
 * with D for each block and T for each tensor computed in the same pass -- the digests to hand to
 * gms_manifest_set_expected.  `image` (device-accessible, written) is device memory or the device
 * view of pinned mapped host memory, as `image_kind` says; bytes of the image that no entry covers
 * are left alone.  Image ranges of different entries must not overlap (GMS_ERR_OVERLAP; restore
 * allows shared sources, capture cannot).  Same kernel as gms_restore with the roles of source and
 * destination exchanged.  Errors: NULL, ALIGN, KIND, OVERLAP, STATE, CUDA.
 */
int gms_capture(const gms_manifest *m, void *image, uint32_t image_kind, uint64_t *d_block_digests,
                uint64_t *d_tensor_digests, void *stream);

/*
 * gms_digest -- Section 3.2 (a replacement engine attaches surviving
 * allocations read-only) and Section 2.2 (reuse only if contents are intact).
 * Same outputs as gms_restore, computed over the destinations where they lie;
 * the destinations are only read.
 */
int gms_digest(const gms_manifest *m, uint64_t *d_block_digests, uint64_t *d_tensor_digests, void *stream);

/*
 * gms_verify -- the trust decision of Section 2.2.  Compares
 * d_block_digests[n_blocks] (device) with the digests recorded by
 * gms_manifest_set_expected and writes the differing (tensor_id, block) pairs
 * to d_out (device, `cap` slots) in ascending (entry position, block) order.
 * *d_count (device, u64) receives the total number of differing blocks, which
 * may exceed cap; only min(count, cap) slots of d_out are written.
 * Errors: NULL, STATE (nothing recorded), CUDA.
 */
int gms_verify(const gms_manifest *m, const uint64_t *d_block_digests, gms_mismatch *d_out, uint32_t cap,
               uint64_t *d_count, void *stream);

/*
 * gms_digest_verify / gms_restore_verify -- gms_digest (resp. gms_restore) followed by gms_verify, with the
 * comparison folded into the pass that computes the digests (Section 2.2 and Section 3.2: the intact-state check
 * sits on the critical path of a reattach, so it should cost no pass of its own).  Outputs are exactly those of
 * the two separate calls: block and tensor digests, the ordered mismatch list and the total count.  While a
 * block's digest is still in a register the streaming kernel compares it with the recorded one and counts the
 * difference against the block's 2048-slot segment; what remains of gms_verify is its ordered emit, one small
 * kernel.  d_block_digests is required here (the emit pass reads it back for the segments that differ).
 * Errors: those of gms_digest / gms_restore, and STATE when nothing has been recorded.
 */
int gms_digest_verify(const gms_manifest *m, uint64_t *d_block_digests, uint64_t *d_tensor_digests, gms_mismatch *d_out,
                      uint32_t cap, uint64_t *d_count, void *stream);
int gms_restore_verify(const gms_manifest *m, const void *image, uint32_t image_kind, uint64_t *d_block_digests,
                       uint64_t *d_tensor_digests, gms_mismatch *d_out, uint32_t cap, uint64_t *d_count, void *stream);

/*
 * gms_verify_tensors -- the per-tensor summary of the same trust decision (Section 2.2): which
 * tensors may be reused as they are.  d_tensor_counts (device, n u32, entry order) receives for
 * every entry the number of its blocks whose digest differs from the recorded one (0 = intact).
 * Errors: NULL, STATE (nothing recorded), CUDA.
 */
int gms_verify_tensors(const gms_manifest *m, const uint64_t *d_block_digests, uint32_t *d_tensor_counts, void *stream);

/*
 * gms_verify_flat_noalloc -- the paper has no counterpart; this is a convenience of this library.
 *
 * Who it is for.  Some callers of a memory service cannot allocate device memory at the moment
 * they need the trust decision: a checker that attaches to a GPU whose memory has already been
 * handed out in full (service slabs plus an engine's KV pool leave no room, so cudaMalloc would
 * fail), or a watchdog that must not enter the allocator because an allocation can stall behind,
 * or disturb, the engine that is serving on the same device.  gms_verify needs a manifest, and
 * building one allocates.  This entry point compares two digest arrays the caller already holds
 * and allocates nothing: no cudaMalloc, no cudaFree, no allocating library call.  Its working
 * table (the per-segment counts of the ordered compaction) lives in a fixed array of about
 * 8 KiB inside the library image, present on every GPU that loads the library until the process
 * exits.
 *
 * What it computes.  Exactly what gms_verify reports for a manifest with the single entry
 * (tensor_id, nbytes = n_blocks * 4096): the pairs (tensor_id, b) with
 * d_computed[b] != d_expected[b], ascending in b, into d_out (device, `cap` slots), and the total
 * number of differing blocks into *d_count (device), which may exceed cap.
 *   d_computed, d_expected  (device) n_blocks u64 each
 *   n_blocks                at most GMS_NOALLOC_MAX_BLOCKS (16 GiB of payload); more is refused
 *                           with GMS_ERR_TOO_LARGE before anything is enqueued
 * Rules.  The first call on a device looks up the device address of the fixed array (a one-time
 * set-up with that device current); make that first call before starting any stream capture.
 * That first call is also when the CUDA runtime loads this library's code and the array onto the
 * device, which itself takes device memory: a caller that expects the GPU to fill up should make
 * one warm-up call with n_blocks <= 16384 and one with n_blocks > 16384 (the two sizes run
 * different kernels) while memory is still available; only calls after that are allocation-free.
 * The cached address does not survive a cudaDeviceReset of that device.
 * All calls on a device share the one array, which keeps the previous call's contents (each call
 * rewrites what it uses before use): two calls that overlap on the GPU race, so keep them on one
 * stream or order them with events.  Errors: NULL, TOO_LARGE, ARG, CUDA.
 */
#define GMS_NOALLOC_MAX_BLOCKS 4194304ull
int gms_verify_flat_noalloc(const uint64_t *d_computed, const uint64_t *d_expected, uint64_t n_blocks, uint64_t tensor_id,
                            gms_mismatch *d_out, uint32_t cap, uint64_t *d_count, void *stream);

/* Device status word of the manifest's last call (synchronises `stream`). 0 = clean; if GMS_DEV_TIMEOUT is
 * set the word is still stored and the call returns GMS_ERR_TIMEOUT (that call's outputs are incomplete). */
int gms_last_device_status(const gms_manifest *m, void *stream, uint64_t *word);

/* A paged KV pool: n_planes planes (layer x {K,V}) of n_blocks blocks. */
#define GMS_KV_IMAGE_BY_ID 1u
typedef struct {
    void *base;            /* (device) 16-byte aligned                                        */
    uint64_t plane_stride; /* bytes between planes, multiple of 16                            */
    uint64_t block_stride; /* bytes between blocks of a plane, multiple of 16, >= block_bytes */
    uint32_t n_planes;
    uint32_t n_blocks;
    uint32_t block_bytes;  /* multiple of 4096, at most 131072                                */
    uint32_t flags;        /* 0, or GMS_KV_IMAGE_BY_ID: the image is pool-shaped -- its slot for
                              list position j is slot d_block_ids[j] (a subset copy between two
                              pools of the same shape) instead of slot j (a packed image)        */
} gms_kv_pool;

/*
 * gms_kv_restore -- Section 6, "Preserving KV state": committed KV blocks
 * kept in host memory or storage are put back after recovery.  For j < n_sel
 * and every plane p:
 *   pool[p][d_block_ids[j]] <- image + p*img_plane_stride + j*img_slot_stride
 * (block_bytes bytes each), with digests
 *   d_block_digests[(j*n_planes + p)*k + c]  for 4 KiB block c of that copy,
 *                                            k = block_bytes/4096;
 *   d_kv_digests[j] = XOR_q mix(D_q ^ q*G), q = p*k + c  (the tensor digest of
 *                                            the slot's planes concatenated).
 * An id outside [0, n_blocks) is skipped: nothing is written to the pool, its
 * digests are 0, and d_status[0] counts it.  With more than one plane,
 * plane_stride must be at least (n_blocks-1)*block_stride + block_bytes
 * (planes that share bytes are refused with GMS_ERR_ARG).  That the image
 * extent covers every slot addressed, and that image and pool do not overlap,
 * is the caller's duty: the library cannot see the size of either buffer.  d_status[1] receives the device
 * status word; d_status[2..3] are scratch for the kernel's work counter.  Ids
 * must be distinct (the caller's duty; duplicates race).
 *   image        (device-accessible) as for gms_restore; strides multiples of 16
 *   d_block_ids  (device) int32[n_sel]
 *   d_block_digests (device) n_sel*n_planes*k u64, may be NULL
 *   d_kv_digests (device) n_sel u64, may be NULL
 *   d_status     (device) 4 u64
 * Errors: NULL, ALIGN, KIND, ARG, CUDA.
 */
int gms_kv_restore(const gms_kv_pool *pool, const void *image, uint64_t img_plane_stride, uint64_t img_slot_stride,
                   uint32_t image_kind, const int32_t *d_block_ids, uint32_t n_sel, uint64_t *d_block_digests,
                   uint64_t *d_kv_digests, uint64_t *d_status, void *stream);

/*
 * gms_kv_capture -- the gather direction of the same extension (Section 6: committed KV blocks are
 * kept in host memory or storage).  pool[p][d_block_ids[j]] is copied into slot j of the packed
 * image for every plane p; arguments, digest layout, skipping of out-of-range ids (the slot is left
 * alone) and status words are those of gms_kv_restore, with `image` written instead of read.
 */
int gms_kv_capture(const gms_kv_pool *pool, void *image, uint64_t img_plane_stride, uint64_t img_slot_stride,
                   uint32_t image_kind, const int32_t *d_block_ids, uint32_t n_sel, uint64_t *d_block_digests,
                   uint64_t *d_kv_digests, uint64_t *d_status, void *stream);

/*
 * gms_kv_digest -- the same extension read together with Section 2.2: KV blocks that outlived an
 * engine may be reused only if they are intact.  pool[p][d_block_ids[j]] is digested where it lies,
 * for every plane p; nothing is written to the pool and there is no image.  Digest layout, skipping
 * of out-of-range ids (digests 0, counted in d_status[0]) and status words are those of
 * gms_kv_restore, so the output compares directly with what gms_kv_restore / gms_kv_capture of the
 * same id list reported (gms_kv_verify names the differing blocks, planes and 4 KiB sub-blocks).
 * pool->flags is ignored apart from the range check.  Errors: NULL, ALIGN, ARG, RANGE, CUDA.
 */
int gms_kv_digest(const gms_kv_pool *pool, const int32_t *d_block_ids, uint32_t n_sel, uint64_t *d_block_digests,
                  uint64_t *d_kv_digests, uint64_t *d_status, void *stream);

/*
 * gms_kv_verify -- the trust decision for preserved KV state (Section 6, "Preserving KV state", read with
 * Section 2.2: state that outlived an engine is reused only if it is intact), in the terms a block manager acts
 * on.  d_computed and d_expected (device, n_sel*n_planes*k u64 each, the layout every gms_kv_* call writes:
 * slot (j*n_planes + p)*k + c) are compared -- typically what gms_kv_digest finds now against what
 * gms_kv_restore / gms_kv_capture reported when the blocks were put back or saved -- and every differing slot is
 * written to d_out (device, `cap` records) as
 *   (block_id = d_block_ids[j], plane = p, sub_block = c, list_pos = j)
 * in ascending (j, p, c) order.  *d_count (device, u64) receives the total, which may exceed cap; only
 * min(count, cap) records are written.  A list position whose id lies outside [0, pool->n_blocks) was skipped by
 * the calls that produced the digests and is never reported, whatever its slots hold.  Only n_planes, n_blocks,
 * block_bytes and flags of `pool` are read.
 *   d_scratch  (device) GMS_KV_VERIFY_SCRATCH_WORDS(n_sel*n_planes*k) u32 of working memory owned by the caller
 *              (the KV calls have no manifest to keep it in); contents before and after are meaningless, and
 *              two calls that overlap on the GPU must not share it
 * Errors: NULL, ALIGN, ARG, RANGE, CUDA.
 */
typedef struct {
    uint32_t block_id;  /* pool block, as given in the id list                        */
    uint32_t plane;     /* layer x {K,V} plane                                        */
    uint32_t sub_block; /* 4 KiB block inside the KV block                            */
    uint32_t list_pos;  /* position of the block in the id list                       */
} gms_kv_mismatch;
#define GMS_KV_VERIFY_SCRATCH_WORDS(n_slots) (((uint64_t)(n_slots) + 2047u) / 2048u + 1u)
int gms_kv_verify(const gms_kv_pool *pool, const int32_t *d_block_ids, uint32_t n_sel, const uint64_t *d_computed,
                  const uint64_t *d_expected, gms_kv_mismatch *d_out, uint32_t cap, uint64_t *d_count, uint32_t *d_scratch,
                  void *stream);

/*
 * Pinned, device-mapped host memory for a GMS_SRC_HOST_MAPPED image (the
 * host-resident snapshot of Section 3.1 step 3 / Section 6).  *device_view is
 * the address to pass as `image`.
 */
int gms_host_image_alloc(uint64_t nbytes, void **host_ptr, void **device_view);
int gms_host_image_free(void *host_ptr);

/*
 * gms_pipe_* / gms_restore_fd -- Section 4, GMS paragraph: with a cold service, a fresh writer
 * fills the model state in from storage while the process is being restored; Section 3.1 prices it
 * at S / B_eff.  The image is read from a file descriptor, never resident as a whole: a ring of
 * `n_buffers` pinned buffers of `buffer_bytes` each (>= 1 MiB, multiple of 4096) is filled by
 * `n_readers` threads with pread(), with a read-ahead hint for the window after (and, after
 * gms_pipe_direct_io(p, 1), bypassing the page cache with O_DIRECT where the file system allows it:
 * right for a cold snapshot on fast storage, wrong for a file the page cache already holds, so it is
 * off unless asked for), and each filled buffer is moved by the
 * copy engine into one of two device buffers of the same size (allocated by gms_pipe_create) and
 * scattered + digested from there by the restore kernel while the next one is read.  If the device
 * buffers cannot be allocated the pipe still works: the kernel then reads the pinned buffers across
 * the host link itself, which reaches about 93 % of what the copy engine does.
 * The first gms_restore_fd (or gms_restore_staged) on a manifest writes a copy of its work list sorted by
 * source offset (on the device, like the other lists) and plans the windows; that call allocates device
 * memory and synchronises, so it must not be made while a stream capture is in progress.  Later calls
 * with the same buffer size reuse the plan.
 * gms_restore_fd is synchronous: on return the stream has been synchronised and the outputs hold
 * exactly what gms_restore would have produced from the same bytes (image byte k = file byte
 * file_offset + k).  One restore at a time per pipe.  Errors: NULL, ARG (bad sizes; a chunk larger
 * than a buffer), NOMEM, STATE, IO (read error or file shorter than the image), CUDA.
 */
typedef struct gms_pipe gms_pipe; /* opaque */
typedef struct {
    uint64_t windows;          /* buffers' worth of image consumed                          */
    uint64_t bytes_read;       /* bytes read from the file                                  */
    double wait_read_seconds;  /* host time spent waiting for readers (storage-bound share) */
    double wait_gpu_seconds;   /* host time spent waiting for a buffer to be released       */
    double total_seconds;      /* wall time of the call                                     */
    uint32_t direct_io;        /* 1: the file system accepted O_DIRECT reads                */
    uint32_t copy_engine;      /* 1: windows went pinned buffer -> copy engine -> device    */
    uint32_t mapped_io;        /* 1: gms_capture_fd stored through a mapping of the file    */
    uint32_t reserved;
} gms_pipe_stats;
int gms_pipe_create(uint32_t n_buffers, uint64_t buffer_bytes, uint32_t n_readers, gms_pipe **out);
int gms_pipe_direct_io(gms_pipe *p, int enable);
int gms_pipe_mapped_writes(gms_pipe *p, int enable);
int gms_pipe_destroy(gms_pipe *p);
int gms_restore_fd(const gms_manifest *m, gms_pipe *p, int fd, uint64_t file_offset, uint64_t *d_block_digests,
                   uint64_t *d_tensor_digests, void *stream, gms_pipe_stats *stats);

/*
 * gms_capture_fd -- the way back through the same pipe: Section 3.1, steps 3 and 4 (device state is staged
 * into host memory and serialised to durable storage).  gms_capture, window by window: the kernel gathers
 * each window of the image straight into one of the pipe's pinned buffers (kernel-issued stores cross the
 * link at the copy engine's rate in this direction, so the device buffers are not used) and the pipe's
 * threads write it out with pwrite() while the next window is gathered.  File byte file_offset + k = image
 * byte k for every byte a tensor covers; bytes of the file between tensors' ranges are not written, and the
 * file is neither truncated nor synced (the caller's fsync decides when it is durable).  Digests as from
 * gms_capture.  `fd` must be open for writing; gms_pipe_direct_io does not apply.  Synchronous like
 * gms_restore_fd; in `stats`, bytes_read counts the bytes written and wait_read_seconds the time spent
 * waiting for the writers.  Errors: NULL, ARG, OVERLAP (tensors share image bytes), NOMEM, STATE, IO
 * (write error), CUDA.
 * gms_pipe_mapped_writes(p, 1): the writers store through a shared mapping of the file instead of calling
 * pwrite().  The kernel lets only one buffered write at a time into a file, so pwrite from many threads
 * runs at one core's copy rate; stores into a mapping run on all of them.  Meant for snapshots kept in
 * the page cache or on tmpfs.  Used only when `fd` is a regular file, open for reading and writing, that
 * already spans file_offset + the image (it is never extended), else pwrite is used as before
 * (stats.mapped_io says which).  The caller must have the file's blocks in that range allocated
 * (written before, or posix_fallocate): a store into a hole of a full file system raises SIGBUS, where
 * pwrite would have returned an error.  Off unless asked for.
 */
int gms_capture_fd(const gms_manifest *m, gms_pipe *p, int fd, uint64_t file_offset, uint64_t *d_block_digests,
                   uint64_t *d_tensor_digests, void *stream, gms_pipe_stats *stats);

/*
 * gms_stage_* / gms_restore_staged -- host-sourced restore with the copy engine on the link
 * (Section 5.2: the existing tool stays far below the PCIe rate; Section 3.1: S / B_eff).  Kernel-issued
 * reads of mapped host memory (gms_restore with GMS_SRC_HOST_MAPPED) top out below what the DMA
 * engine reaches on the same link.  Here the pinned host image is moved window by window with
 * cudaMemcpyAsync on an internal stream into a ring of `n_buffers` device buffers of `buffer_bytes`
 * each (>= 1 MiB, multiple of 4096), and every landed window is scattered and digested by the
 * restore kernel on the caller's stream while the next one is in flight; all ordering is done with
 * stream events, no kernel waits for a flag.  Asynchronous like gms_restore (after the first call on a
 * manifest, which uploads the sorted work list as described above): outputs are valid once
 * `stream` has been synchronised; the host image must stay untouched until then.  Results are
 * exactly those of gms_restore from the same bytes.  `host_image` (host) must be pinned memory.
 * Errors: NULL, ARG, KIND (not pinned host memory), NOMEM, STATE, CUDA.
 */
typedef struct gms_stage gms_stage; /* opaque */
int gms_stage_create(uint32_t n_buffers, uint64_t buffer_bytes, gms_stage **out);
int gms_stage_destroy(gms_stage *st);
int gms_restore_staged(const gms_manifest *m, gms_stage *st, const void *host_image, uint64_t *d_block_digests,
                       uint64_t *d_tensor_digests, void *stream);

/*
 * gms_service_* -- the substrate under the destinations: Section 4, GMS paragraph (physical
 * allocations made with cuMemCreate, a first-fit suballocator over 2 GiB slabs with dedicated
 * slabs for larger allocations, permissions set per slab) and Section 3.2 (ownership protocol:
 * EMPTY -> RW, one writer populates -> COMMITTED, immutable -> RO while n >= 1 readers hold it;
 * a writer that gives up before commit discards everything; write access returns after the last
 * reader has left; read-only is enforced with cuMemSetAccess).  Current device.  The state machine
 * lives in the process that created the service; other processes take part through the export / import
 * calls further down.
 *   create      slab_bytes = 0 means 2 GiB; GMS_SERVICE_DRY_RUN keeps the books without any CUDA
 *               call (addresses are made up and must not be dereferenced)
 *   acquire_rw  EMPTY -> RW, or COMMITTED -> RW (contents and addresses kept, slabs writable again);
 *               GMS_ERR_STATE while a writer or readers hold the service
 *   alloc       RW only; 256-byte aligned device address, first fit over the slabs, a dedicated slab
 *               if nbytes exceeds the slab size; individual allocations are never freed, only all
 *               at once (abort / destroy)
 *   commit      RW -> COMMITTED: the device is synchronised, then every slab becomes read-only
 *   abort       RW -> EMPTY: every slab is unmapped and released
 *   acquire_ro / release_ro   COMMITTED <-> RO with a reader count
 * After commit the addresses may be read by anything (gms_digest, gms_capture, an engine's
 * kernels); writing to them faults the writing context, so gms_restore / gms_kv_restore must only
 * target them in state RW (gms_service_access tells which it is).  Errors: NULL, ARG, STATE, NOMEM,
 * RANGE (access: not an address of this service), CUDA.
 */
#define GMS_STATE_EMPTY 0u
#define GMS_STATE_RW 1u
#define GMS_STATE_COMMITTED 2u
#define GMS_STATE_RO 3u
#define GMS_SERVICE_DRY_RUN 1u
#define GMS_SERVICE_SHAREABLE 2u /* slabs can be handed to other processes (gms_service_export_fd) */
typedef struct gms_service gms_service; /* opaque */
typedef struct {
    uint32_t state, readers;
    uint64_t n_slabs, n_dedicated; /* slabs in all, and those holding one oversized allocation */
    uint64_t slab_bytes;           /* regular slab size after rounding to the mapping granularity */
    uint64_t bytes_reserved;       /* sum of slab sizes                                           */
    uint64_t bytes_allocated;      /* sum of (256-byte rounded) allocation sizes                  */
    uint32_t attached;             /* 0 between gms_service_detach and gms_service_reattach        */
    uint32_t backed;               /* 0 between gms_service_release_pages and gms_service_back_pages */
} gms_service_stats;
int gms_service_create(uint64_t slab_bytes, uint32_t flags, gms_service **out);
int gms_service_destroy(gms_service *s);
int gms_service_acquire_rw(gms_service *s);
int gms_service_alloc(gms_service *s, uint64_t nbytes, void **dptr);
int gms_service_commit(gms_service *s);
int gms_service_abort(gms_service *s);
int gms_service_acquire_ro(gms_service *s);
int gms_service_release_ro(gms_service *s);
int gms_service_info(gms_service *s, gms_service_stats *out);
int gms_service_access(gms_service *s, const void *dptr, uint32_t *writable);

/*
 * Addresses that outlive their mappings.  A snapshot of an engine holds the virtual addresses of its
 * tensors (in CUDA graphs and tensor metadata) but none of the memory behind them, so both calls
 * below keep every virtual range reserved: the destination pointers of a manifest built before
 * stay valid afterwards.
 *   detach / reattach           Section 3.3: before capture the engine unmaps each service range but
 *       keeps its address reservation while the service keeps the physical memory; after restore the
 *       surviving memory is mapped read-only at the same addresses.  COMMITTED (no readers) only.
 *       Between the two calls nothing may touch the addresses (gms_service_access returns
 *       GMS_ERR_STATE) and acquire_rw / acquire_ro are refused.  Contents are preserved.
 *   release_pages / back_pages  Section 3.1 (pages released before capture, fresh pages mapped at the
 *       same addresses after restore) and Section 3.3 (after a device-invalidating failure the state
 *       is rebuilt in fresh allocations): RW only.  The physical memory of every slab is given back
 *       to the driver; back_pages maps fresh memory, writable, whose contents are undefined until the
 *       writer restores them (gms_restore, gms_kv_restore).  In between, alloc / commit are refused.
 * Both pairs synchronise the device first.  Errors: NULL, STATE, NOMEM (back_pages; the service then
 * stays without pages), CUDA.
 */
int gms_service_detach(gms_service *s);
int gms_service_reattach(gms_service *s);
int gms_service_release_pages(gms_service *s);
int gms_service_back_pages(gms_service *s);

/*
 * Across processes -- Section 4, GMS paragraph (the service process creates the physical allocations and
 * keeps their handles; clients receive them as file descriptors over Unix sockets, import them, map them and
 * set their own access) and Section 3.2 (the memory therefore outlives the engine process that filled or used
 * it, and the replacement engine attaches it read-only).  The library provides the two ends; the socket and
 * whatever is said on it (who holds the service in which state) belong to the processes that use them.
 *   gms_service_slab       size and address of slab `index` (0 .. n_slabs-1 of gms_service_info) in the service's
 *                          own address space, so that allocation addresses can be written as (slab, offset)
 *   gms_service_export_fd  a new file descriptor for slab `index` (service created with GMS_SERVICE_SHAREABLE;
 *                          GMS_ERR_STATE otherwise, in a dry run, or without pages); the caller sends it with
 *                          SCM_RIGHTS and closes its copy.  The memory lives as long as any process holds a
 *                          handle or a mapping of it.
 *   gms_import_create      the client's side, on the same GPU (the current device): imports the n descriptors
 *                          (which stay open; the caller closes them), reserves address space for each -- at
 *                          slabs[i].address where that is free -- maps it and sets this process's access:
 *                          read-only, or writable with GMS_IMPORT_WRITABLE (the writer that populates, RW in the
 *                          protocol).  GMS_IMPORT_SAME_ADDRESS: fail with GMS_ERR_RANGE unless every slab lands
 *                          at the service's address (an engine restored from a snapshot has those addresses in its
 *                          graphs and metadata, and kept the ranges free; a fresh process will often find them
 *                          taken); without it any address will do and gms_import_address tells which.  Permissions are per process: a reader's mapping stays read-only whatever the
 *                          others hold.
 *   gms_import_destroy     synchronises the device, unmaps, frees the address ranges and drops the handles; the
 *                          contents stay with the service.
 * Errors: NULL, ARG, RANGE, STATE, NOMEM, CUDA.
 */
#define GMS_IMPORT_WRITABLE 1u
#define GMS_IMPORT_SAME_ADDRESS 2u
typedef struct {
    uint64_t address, bytes;
    uint32_t dedicated, reserved;
} gms_slab_info;
typedef struct gms_import gms_import; /* opaque */
int gms_service_slab(gms_service *s, uint64_t index, gms_slab_info *out);
int gms_service_export_fd(gms_service *s, uint64_t index, int *fd);
int gms_import_create(const int *fds, const gms_slab_info *slabs, size_t n, uint32_t flags, gms_import **out);
int gms_import_address(const gms_import *imp, size_t index, void **dptr);
int gms_import_destroy(gms_import *imp);

/*
 * Tuning and test hooks.  The library reads the environment variables below once per process (the chunk lengths
 * once per gms_manifest_build), and ONLY if GMS_TUNING_HOOKS=1 is set as well; without that switch none of them has
 * any effect, so a stray variable in a serving process cannot change launch shapes or chunking.  Every setting
 * gives bit-identical results (the test suite runs the parity checks under several of them); the defaults are what
 * the published timings were taken with.
 *   GMS_GEOM_RESTORE / GMS_GEOM_DIGEST / GMS_GEOM_KV   "warps,slots,CTAs-per-SM" of the restore/capture kernel, the
 *       digest-only kernels and the KV copy kernels (defaults 9,4,1 / 16,3,1 / 8,6,1; warps 1..16, slots 3|4|6|8)
 *   GMS_CLAIM_RESTORE / GMS_CLAIM_DIGEST               "counters,chunks-per-claim" of the work-list claims
 *       (defaults 1,1 / 2,1; counters 1..32, chunks 1..64)
 *   GMS_CHUNK_BLOCKS / GMS_CHUNK_BLOCKS_DIGEST         4 KiB blocks per chunk of the copy list and of the digest
 *       list (defaults 4 / 8, fewer for small manifests; 1..32)
 *   GMS_L2_KEEP                                        0 / 1: never / always give the digest-only kernels their L2
 *       hints (payload loads evict-first, digest stores evict-last); by default they are used for payloads from
 *       256 MiB on whose digests take at most 16 MiB
 *   GMS_CHECK_TABLES                                   1: gms_manifest_build reads the work lists it wrote on the
 *       device back and compares them with a host construction of the same lists (GMS_ERR_STATE if they differ)
 */

/* Launch geometry of the streaming kernels on the current device (for reporting). */
int gms_launch_geometry(uint32_t *grid_ctas, uint32_t *warps_per_cta, uint32_t *smem_bytes);
/* Number of kernels this library has launched in this process so far (for reporting). */
uint64_t gms_kernel_launches(void);
/*
 * Makes `device` current for the calling thread's later gms_* calls.  The library links its own
 * copy of the CUDA runtime; a process that drives several GPUs (one service per GPU, Section 4)
 * selects the device here as well as in whatever else it uses.
 */
int gms_set_device(int device);

const char *gms_strerror(int status);
const char *gms_last_cuda_error(void); /* text of the last failed CUDA call on this thread */
uint32_t gms_version(void);

#ifdef __cplusplus
}
#endif
#endif /* GMS_H */
