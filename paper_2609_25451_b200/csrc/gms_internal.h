// Internal declarations shared by the host API and the kernel translation units.
// Nothing here is part of the public ABI (that is include/gms.h).
#pragma once
#include <cstddef>
#include <cstdint>
#include <cstdio>
#include <cstdlib>
#include <utility>
#include <vector>

#include <cuda_runtime.h>

namespace gms {

constexpr uint32_t kBlockBytes = 4096;     // digest block
constexpr uint32_t kMaxChunkBlocks = 32;   // one lane keeps one block digest of the chunk in flight
constexpr uint64_t kG = 0x9E3779B97F4A7C15ull;
constexpr uint32_t kMaxCounters = 32;      // work counters a manifest carries
constexpr uint32_t kCounterStride = 64;    // 32-bit words between counters (256 B: separate L2 lines)

// One unit of the persistent kernels' work list: a run of whole digest blocks of
// one tensor (the last block of a tensor may be short).  32 bytes, read as 2 x 16 B.
struct alignas(16) Chunk {
    uint64_t src_off;  // byte offset of the run in the packed image
    uint64_t dst;      // device address of the run in its destination
    uint32_t nbytes;   // 1 .. kMaxChunkBlocks * 4096
    uint32_t tensor;   // entry index (slot of the tensor digest)
    uint32_t gblock0;  // slot of the run's first block digest
    uint32_t tblock0;  // index of that block inside the tensor
};
static_assert(sizeof(Chunk) == 32, "Chunk must stay 32 bytes");

// Launch shape of the streaming kernels (chosen once per process, per device).
struct Geometry {
    uint32_t grid;     // CTAs (a multiple of the SM count)
    uint32_t warps;    // warps per CTA; every warp runs its own copy pipeline
    uint32_t stages;   // 4 KiB ring slots per warp
    uint32_t smem;     // dynamic shared memory per CTA
    uint32_t counters; // work counters the chunk claims are spread over
    uint32_t group;    // consecutive chunks bought by one claim
};
enum Kind { kRestore = 0, kDigest = 1, kKv = 2, kKvDigest = 3, kKinds = 4 };  // each streaming kernel has its own shape
cudaError_t get_geometry(Kind kind, Geometry *g);

struct StreamArgs {
    const Chunk *chunks;
    uint32_t n_chunks;
    const uint8_t *image;          // restore: base of the packed image; digest: unused
    uint64_t *block_digests;       // may be null
    uint64_t *tensor_digests;      // may be null
    uint32_t n_tensors;
    unsigned int *work_counters;   // manifest-owned: kMaxCounters counters, kCounterStride words apart
    unsigned long long *status;    // manifest-owned device status word
    uint32_t n_counters;           // filled in by the launcher
    uint32_t group;                // filled in by the launcher
    uint32_t capture;              // 1: gather allocations into the image (restore kernel with roles swapped)
    uint32_t keep_accum;           // 1: a later window of a windowed restore (accumulators and status are kept)
    uint32_t stall_chunk;          // self-test (GMS_BUILD_SELFTEST_STALL): chunk whose first wait runs out; else 0xffffffff
    const uint64_t *expected;      // fused compare: the recorded block digests (null: no compare)
    uint32_t *seg_count;           // fused compare: per-segment mismatch counters, cleared by the prologue
    uint32_t n_segments;
    uint32_t l2_keep;              // digest-only kernel: 1 = L2 hints on (see kL2KeepBytes)
};

// The digest-only kernels write 8 bytes per 4 KiB they read.  When that output is small next to the L2 (126 MB),
// it pays to keep it there for the length of the kernel and let the payload, which is read once, go first: the
// bulk loads carry an evict-first hint and the digest stores an evict-last one.  Dirty digest lines that trickle
// out to DRAM one by one in the middle of a read stream cost far more than their bytes (measured with the output
// confined to 64 KiB: 2.16 against 2.21 ms on a 16 GB manifest), and with the hints the 12 MB of the 60 GB KV
// pool's digests stay put (0.861 -> 0.843 ms; mixed manifest, 4 MB: 0.339 -> 0.333 ms).  A 31 MB output measured
// no better with the hints than without (2.206 / 2.208 ms), and the copying kernels measured slower with them
// (4.72 -> 4.79 ms), so they are used by the digest-only kernels alone, and only below this output size.  Nor
// for a payload that the L2 could hold itself: marking it evict-first costs the call that comes next (tiny
// manifest, 34 MB: the restore behind the digest pass 22.4 -> 23.2 us).  The price: after such a call up to
// 16 MiB of digest lines sit in L2 at the higher retention priority until the cache replaces them (it is a
// replacement hint, not a reservation: nothing is pinned and nothing has to be reset).
constexpr uint64_t kL2KeepBytes = 16ull << 20;
constexpr uint64_t kL2KeepMinBlocks = (256ull << 20) / kBlockBytes;  // payloads from 256 MiB on (twice the L2)
uint32_t l2_keep_for(uint64_t n_blocks);  // 1 if a digest-only pass over n_blocks blocks gets the hints (hook: GMS_L2_KEEP)

struct KvArgs {
    uint8_t *pool_base;
    uint64_t plane_stride, block_stride;
    uint32_t n_planes, n_blocks, block_bytes;
    const uint8_t *image;
    uint64_t img_plane_stride, img_slot_stride;
    const int32_t *ids;
    uint32_t n_sel;
    uint64_t *block_digests;       // may be null
    uint64_t *kv_digests;          // may be null
    unsigned long long *status;    // [0] skipped ids, [1] device status word, [2] work counter, [3] spare
    uint32_t capture;              // 1: gather pool blocks into the image
    uint32_t digest_only;          // 1: digest the selected pool blocks where they lie (no image, nothing written)
    uint32_t by_id;               // 1: the image is pool-shaped (slot = block id), else packed (slot = list position)
    uint32_t l2_keep;              // digest-only: 1 = L2 hints on (see kL2KeepBytes)
};

cudaError_t launch_restore(const StreamArgs &a, cudaStream_t s);
cudaError_t launch_digest(const StreamArgs &a, cudaStream_t s);
cudaError_t launch_kv_restore(const KvArgs &a, cudaStream_t s);

struct VerifyArgs {
    const uint64_t *computed, *expected;
    uint64_t n_blocks;
    const uint64_t *block_base;    // n_tensors + 1 prefix sums (device)
    const uint64_t *tensor_ids;    // n_tensors (device)
    uint32_t n_tensors;
    uint32_t *seg_count;           // n_segments scratch (device): differing slots per segment
    uint32_t n_segments;
    void *out;                     // gms_mismatch[cap] (gms_kv_mismatch[cap] in KV mode)
    uint32_t cap;
    uint64_t *count;
    // KV mode (gms_kv_verify): slots are [list position][plane][sub-block]; 0 slots per id = manifest mode
    const int32_t *kv_ids;
    uint32_t kv_slots_per_id;      // n_planes * (block_bytes / 4096)
    uint32_t kv_k;                 // block_bytes / 4096
    uint32_t kv_pool_blocks;       // ids outside [0, kv_pool_blocks) are never reported
};
constexpr uint32_t kVerifySegShift = 11;
constexpr uint32_t kVerifySegBlocks = 1u << kVerifySegShift;  // digest slots compared by one CTA (one counter each)
cudaError_t launch_verify(const VerifyArgs &a, cudaStream_t s);
// scan + emit only: the per-segment counts have been produced by a streaming kernel's fused compare
cudaError_t launch_verify_counted(const VerifyArgs &a, cudaStream_t s);
cudaError_t launch_verify_tensor_counts(const VerifyArgs &a, uint32_t *counts, cudaStream_t s);
cudaError_t launch_copy_u64(uint64_t *dst, const uint64_t *src, uint64_t n, cudaStream_t s);

// Expansion of the layout record into one chunk list on the device (gms_build_kernels.cu).  All pointers are device
// memory; the per-tensor columns are the record's fields, full_base the prefix sums of full-length chunks per tensor,
// tail_pos the list position of each tensor's short last chunk (0xffffffff: it has none).
struct ExpandArgs {
    const uint64_t *src_offset, *dst, *nbytes;  // n_tensors each
    const uint64_t *block_base;                 // n_tensors + 1
    const uint64_t *full_base;                  // n_tensors + 1
    const uint32_t *tail_pos;                   // n_tensors
    const uint32_t *perm;                       // null, or n_tensors: list slot -> entry index (lists in another tensor order;
                                                // full_base and tail_pos are then indexed by slot, the columns by entry)
    uint32_t n_tensors;
    uint64_t n_full;
    uint32_t chunk_blocks;
    Chunk *out;
};
cudaError_t launch_expand_chunks(const ExpandArgs &a, cudaStream_t s);

// A window of a restore that is fed piecewise (file -> pinned buffer -> device): a run of the
// chunk list sorted by source offset whose sources all lie in image bytes [src_lo, src_hi).
struct SrcWindow {
    uint32_t first_chunk, n_chunks;
    uint64_t src_lo, src_hi;
};

void count_launches(uint32_t n);  // bumps the process-wide launch counter
int report_cuda_error(cudaError_t e);  // records the text for gms_last_cuda_error(); returns GMS_ERR_CUDA

}  // namespace gms

struct gms_manifest;
namespace gms {
// Cuts the manifest's work into windows of at most `buffer_bytes` of image each (building, once,
// a device copy of the chunk list sorted by source offset).  Returns a GMS_* status.
int manifest_src_windows(const gms_manifest *m, uint64_t buffer_bytes, std::vector<SrcWindow> *out);
// Enqueues the restore of one window; `window_base` is the device-accessible address of image byte w.src_lo.
// With `capture` the window is written instead (allocations -> window), by the same kernel.
int manifest_launch_window(const gms_manifest *m, const SrcWindow &w, const void *window_base, bool first,
                           uint64_t *d_block_digests, uint64_t *d_tensor_digests, cudaStream_t s, bool capture = false);
// The image ranges (offset, length) of the non-empty tensors in ascending order of offset; GMS_ERR_OVERLAP if two
// tensors share image bytes.
int manifest_sorted_sources(const gms_manifest *m, std::vector<std::pair<uint64_t, uint64_t>> *out);
uint64_t manifest_n_tensors(const gms_manifest *m);
}  // namespace gms
