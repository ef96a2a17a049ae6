// gms_verify: compare computed block digests with the recorded ones and emit
// the differing (tensor_id, block) pairs in ascending (entry position, block)
// order.  The order is made deterministic by an ordered compaction instead of
// an atomic append: (1) every CTA counts the differences in its own contiguous
// segment of 2048 digest slots (or a streaming kernel has already counted them
// while it held each digest in a register: the fused compare), (2) every CTA
// whose segment has differences (normally none) adds up the counts of the
// segments before it -- a few kilobytes out of L2 -- ranks its own differences
// with a block-wide scan and writes them at offset + rank; the last CTA also
// writes the grand total.  Traffic is 16 bytes per 4 KiB of payload -- noise
// next to the streaming kernels -- and no CTA ever waits for another.
// Every kernel here may be scheduled while its predecessor on the stream still
// runs (programmatic dependent launch) and waits for it before reading.
#include "gms_internal.h"

namespace gms {
namespace {

constexpr uint32_t kThreads = 256;
constexpr uint32_t kPerThread = kVerifySegBlocks / kThreads;  // 8 consecutive slots per thread
static_assert(kVerifySegBlocks % kThreads == 0, "segment must divide evenly");

struct Mismatch {
    uint64_t tensor_id, block;
};

// Whether a differing slot counts.  Manifest mode: always.  KV mode (gms_kv_verify): only if the slot belongs to a
// list position whose block id lies inside the pool -- an id outside it was skipped by the call that produced the
// digests and is never reported.
template <bool kKv>
__device__ __forceinline__ bool counts(const VerifyArgs &a, uint64_t g)
{
    if (!kKv) return true;
    const int32_t id = a.kv_ids[g / a.kv_slots_per_id];
    return id >= 0 && (uint32_t)id < a.kv_pool_blocks;
}

template <bool kKv>
__device__ __forceinline__ uint32_t diff_mask(const VerifyArgs &a, uint64_t first)
{
    uint32_t mask = 0;
#pragma unroll
    for (uint32_t k = 0; k < kPerThread; ++k) {
        const uint64_t g = first + k;
        if (g < a.n_blocks && a.computed[g] != a.expected[g] && counts<kKv>(a, g)) mask |= 1u << k;
    }
    return mask;
}

// One output record for differing slot g.  Manifest mode: (tensor_id, block inside the tensor), found by binary
// search of the block-base table.  KV mode: slots are laid out [list position j][plane][4 KiB sub-block], and the
// record is (block id, plane, sub-block, j).
template <bool kKv>
__device__ __forceinline__ void write_record(const VerifyArgs &a, uint64_t rank, uint64_t g)
{
    if (kKv) {
        const uint32_t j = (uint32_t)(g / a.kv_slots_per_id), r = (uint32_t)(g % a.kv_slots_per_id);
        static_cast<uint4 *>(a.out)[rank] = make_uint4((uint32_t)a.kv_ids[j], r / a.kv_k, r % a.kv_k, j);
        return;
    }
    // entry t with block_base[t] <= g < block_base[t+1]; empty tensors share a base and are skipped
    uint32_t lo = 0, hi = a.n_tensors;
    while (hi - lo > 1) {
        const uint32_t mid = lo + (hi - lo) / 2;
        if (a.block_base[mid] <= g) lo = mid; else hi = mid;
    }
    Mismatch *out = static_cast<Mismatch *>(a.out);
    out[rank].tensor_id = a.tensor_ids[lo];
    out[rank].block = g - a.block_base[lo];
}

template <bool kKv>
__global__ void __launch_bounds__(kThreads) gms_verify_count_kernel(VerifyArgs a)
{
    asm volatile("griddepcontrol.launch_dependents;");  // the emit kernel may be scheduled; it waits for our counts
    asm volatile("griddepcontrol.wait;" ::: "memory");  // the digests being compared are complete and visible
    __shared__ uint32_t warp_sum[kThreads / 32];
    // only the segment's total matters here, so the slots are read coalesced (16-byte pairs, neighbouring lanes
    // neighbouring pairs); the emit pass, which needs ranks, uses the thread-contiguous layout
    const uint64_t seg0 = (uint64_t)blockIdx.x * kVerifySegBlocks;
    const bool vec = ((reinterpret_cast<uint64_t>(a.computed) | reinterpret_cast<uint64_t>(a.expected)) & 15u) == 0;
    uint32_t c = 0;
#pragma unroll
    for (uint32_t k = 0; k < kPerThread / 2; ++k) {
        const uint64_t g = seg0 + 2ull * (k * kThreads + threadIdx.x);
        if (vec && g + 1 < a.n_blocks) {
            const ulonglong2 p = *reinterpret_cast<const ulonglong2 *>(a.computed + g);
            const ulonglong2 q = *reinterpret_cast<const ulonglong2 *>(a.expected + g);
            c += (p.x != q.x && counts<kKv>(a, g)) + (p.y != q.y && counts<kKv>(a, g + 1));
        } else {  // arrays that are only 8-byte aligned, and the odd last slot
            if (g < a.n_blocks) c += a.computed[g] != a.expected[g] && counts<kKv>(a, g);
            if (g + 1 < a.n_blocks) c += a.computed[g + 1] != a.expected[g + 1] && counts<kKv>(a, g + 1);
        }
    }
    c = __reduce_add_sync(0xffffffffu, c);
    if ((threadIdx.x & 31) == 0) warp_sum[threadIdx.x >> 5] = c;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t t = 0;
        for (uint32_t w = 0; w < kThreads / 32; ++w) t += warp_sum[w];
        a.seg_count[blockIdx.x] = t;
    }
}

// Ordered emit.  CTA k owns segment k.  Its offset in the output is the sum of the counts of segments 0..k-1,
// which it adds up itself (at most a few thousand 32-bit words, read by 256 threads); segments without
// differences return at once, except the last one, which also publishes the total.
template <bool kKv>
__global__ void __launch_bounds__(kThreads) gms_verify_emit_kernel(VerifyArgs a)
{
    asm volatile("griddepcontrol.launch_dependents;");
    asm volatile("griddepcontrol.wait;" ::: "memory");  // the per-segment counts are complete and visible
    __shared__ uint64_t warp_tot[kThreads / 32];
    __shared__ uint32_t warp_sum[kThreads / 32];
    if (a.n_segments == 0) {  // no digest slots at all
        if (threadIdx.x == 0) *a.count = 0;
        return;
    }
    const bool last = blockIdx.x + 1 == a.n_segments;
    const uint32_t own = a.seg_count[blockIdx.x];
    if (own == 0 && !last) return;  // the common case: nothing differs here
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint64_t before = 0;
    for (uint32_t i = threadIdx.x; i < blockIdx.x; i += kThreads) before += a.seg_count[i];
#pragma unroll
    for (int d = 16; d; d >>= 1) before += __shfl_xor_sync(0xffffffffu, before, d);
    if (lane == 0) warp_tot[warp] = before;
    __syncthreads();
    before = 0;
    for (uint32_t w = 0; w < kThreads / 32; ++w) before += warp_tot[w];
    if (last && threadIdx.x == 0) *a.count = before + own;
    if (own == 0) return;
    const uint64_t first = (uint64_t)blockIdx.x * kVerifySegBlocks + (uint64_t)threadIdx.x * kPerThread;
    const uint32_t mask = diff_mask<kKv>(a, first);
    const uint32_t mine = __popc(mask);
    uint32_t incl = mine;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t o = __shfl_up_sync(0xffffffffu, incl, d);
        if ((int)lane >= d) incl += o;
    }
    if (lane == 31) warp_sum[warp] = incl;
    __syncthreads();
    uint64_t rank = before + incl - mine;
    for (uint32_t w = 0; w < warp; ++w) rank += warp_sum[w];
    if (!mask) return;
    for (uint32_t k = 0; k < kPerThread; ++k) {
        if (!(mask & (1u << k))) continue;
        if (rank < a.cap) write_record<kKv>(a, rank, first + k);
        ++rank;
    }
}

// Small inputs (a few thousand digest slots): the three passes in one CTA, one launch.
constexpr uint32_t kSmallThreads = 1024;
constexpr uint64_t kSmallBlocks = 16384;
template <bool kKv>
__global__ void __launch_bounds__(kSmallThreads) gms_verify_small_kernel(VerifyArgs a)
{
    __shared__ uint32_t warp_sum[kSmallThreads / 32];
    asm volatile("griddepcontrol.launch_dependents;");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const uint64_t per = (a.n_blocks + kSmallThreads - 1) / kSmallThreads;  // consecutive slots per thread
    const uint64_t lo = (uint64_t)threadIdx.x * per, hi = lo + per < a.n_blocks ? lo + per : a.n_blocks;
    uint32_t mine = 0;
    for (uint64_t g = lo; g < hi; ++g) mine += a.computed[g] != a.expected[g] && counts<kKv>(a, g);
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t incl = mine;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t o = __shfl_up_sync(0xffffffffu, incl, d);
        if ((int)lane >= d) incl += o;
    }
    if (lane == 31) warp_sum[warp] = incl;
    __syncthreads();
    uint64_t rank = incl - mine, total = 0;
    for (uint32_t w = 0; w < kSmallThreads / 32; ++w) {
        if (w < warp) rank += warp_sum[w];
        total += warp_sum[w];
    }
    if (threadIdx.x == 0) *a.count = total;
    if (!mine) return;
    for (uint64_t g = lo; g < hi; ++g) {
        if (a.computed[g] == a.expected[g] || !counts<kKv>(a, g)) continue;
        if (rank < a.cap) write_record<kKv>(a, rank, g);
        ++rank;
    }
}

__global__ void gms_copy_u64_kernel(uint64_t *dst, const uint64_t *src, uint64_t n)
{
    asm volatile("griddepcontrol.launch_dependents;");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const uint64_t step = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += step) dst[i] = src[i];
}

}  // namespace

namespace {
template <class... P, class... A>
cudaError_t launch_pdl(void (*kernel)(P...), dim3 grid, dim3 block, cudaStream_t s, A... args)
{
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.stream = s;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}
}  // namespace

cudaError_t launch_verify_counted(const VerifyArgs &a, cudaStream_t s)
{
    count_launches(1);
    const dim3 grid(a.n_segments ? a.n_segments : 1);
    return a.kv_slots_per_id ? launch_pdl(gms_verify_emit_kernel<true>, grid, dim3(kThreads), s, a)
                             : launch_pdl(gms_verify_emit_kernel<false>, grid, dim3(kThreads), s, a);
}

cudaError_t launch_verify(const VerifyArgs &a, cudaStream_t s)
{
    const bool kv = a.kv_slots_per_id != 0;
    if (a.n_segments == 0) return launch_verify_counted(a, s);  // no digest slots at all: count = 0
    if (a.n_blocks <= kSmallBlocks) {
        count_launches(1);
        return kv ? launch_pdl(gms_verify_small_kernel<true>, dim3(1), dim3(kSmallThreads), s, a)
                  : launch_pdl(gms_verify_small_kernel<false>, dim3(1), dim3(kSmallThreads), s, a);
    }
    count_launches(1);
    cudaError_t e = kv ? launch_pdl(gms_verify_count_kernel<true>, dim3(a.n_segments), dim3(kThreads), s, a)
                       : launch_pdl(gms_verify_count_kernel<false>, dim3(a.n_segments), dim3(kThreads), s, a);
    if (e) return e;
    return launch_verify_counted(a, s);
}

namespace {

// Per-tensor summary: counts[t] = number of differing blocks of entry t.  One warp per tensor-sized slice
// would be badly balanced (1 .. 262,144 blocks per tensor), so the slots are walked grid-stride and the rare
// differing slot looks its tensor up and bumps that counter.
__global__ void gms_verify_tensor_counts_kernel(VerifyArgs a, uint32_t *counts)
{
    asm volatile("griddepcontrol.launch_dependents;");
    asm volatile("griddepcontrol.wait;" ::: "memory");  // the zeroed counters and the digests are visible
    const uint64_t step = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t g = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; g < a.n_blocks; g += step) {
        if (a.computed[g] == a.expected[g]) continue;
        uint32_t lo = 0, hi = a.n_tensors;
        while (hi - lo > 1) {
            const uint32_t mid = lo + (hi - lo) / 2;
            if (a.block_base[mid] <= g) lo = mid; else hi = mid;
        }
        atomicAdd(counts + lo, 1u);
    }
}

__global__ void gms_zero_u32_kernel(uint32_t *p, uint64_t n)
{
    asm volatile("griddepcontrol.launch_dependents;");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const uint64_t step = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += step) p[i] = 0;
}

}  // namespace

cudaError_t launch_verify_tensor_counts(const VerifyArgs &a, uint32_t *counts, cudaStream_t s)
{
    if (a.n_tensors == 0) return cudaSuccess;
    uint32_t zb = (a.n_tensors + 255) / 256;
    cudaError_t e = launch_pdl(gms_zero_u32_kernel, dim3(zb > 592 ? 592 : zb), dim3(256), s, counts, (uint64_t)a.n_tensors);
    if (e) return e;
    count_launches(1);
    if (a.n_blocks == 0) return cudaSuccess;
    uint64_t blocks = (a.n_blocks + 1023) / 1024;
    if (blocks > 148 * 8) blocks = 148 * 8;
    count_launches(1);
    return launch_pdl(gms_verify_tensor_counts_kernel, dim3((uint32_t)blocks), dim3(256), s, a, counts);
}

cudaError_t launch_copy_u64(uint64_t *dst, const uint64_t *src, uint64_t n, cudaStream_t s)
{
    if (n == 0) return cudaSuccess;
    uint64_t blocks = (n + 1023) / 1024;
    if (blocks > 148 * 8) blocks = 148 * 8;
    count_launches(1);
    return launch_pdl(gms_copy_u64_kernel, dim3((uint32_t)blocks), dim3(256), s, dst, src, n);
}

}  // namespace gms
