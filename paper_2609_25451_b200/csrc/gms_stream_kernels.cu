// Persistent streaming kernels of the restore / digest path (sm_100a).
//
// Shape of the work.  A restore is HBM-bound: every payload byte is read once
// and written once, and the digest costs ~17 integer instructions per 8-byte
// word, which fits under the memory time.  Nothing here is a contraction, so
// no tensor cores; what matters is bytes in flight, full-line transactions and
// no per-tensor launches.
//
// Design.  One CTA per SM, a dozen warps per CTA, and every warp is its own
// small pipeline with no CTA-wide synchronisation at all:
//   * the warp claims a chunk (<= 32 digest blocks of one tensor) from the
//     manifest's work list with one atomicAdd -- no warp ever waits for another;
//   * lane 0 moves each 4 KiB digest block with a 1-D bulk async copy (TMA)
//     global -> shared, completion signalled on an mbarrier, up to S-1 blocks
//     ahead of the block being digested (S ring slots per warp);
//   * when a block has landed, lane 0 sends it on its way to the destination
//     with a bulk copy shared -> global straight from the same slot (the payload
//     never passes through registers), while all 32 lanes read the slot with
//     16-byte shared loads and fold it into the block digest;
//   * the 32 lane partials are XOR-reduced with redux.sync; each lane keeps the
//     digest of one block of the chunk, so that at the end of the chunk the
//     block digests leave as one coalesced store and the chunk's share of the
//     tensor digest as a single 64-bit atomicXor.
// XOR makes every result independent of which warp did what, in which order.
//
// Two exact rewrites of mix() keep the instruction count down (both are
// bit-identical to the definition, which the CPU oracle follows literally):
//   (z ^ (z >> 30)) with z = w ^ c equals (w ^ (w >> 30)) ^ (c ^ (c >> 30)), so
//     the per-position constant is folded and held in registers (each lane
//     always sees the same 16 word positions of a block);
//   the last step y ^ (y >> 31) is linear over XOR, so it is applied once to
//     the XOR of the 512 partial values instead of 512 times.
//
// Every wait is bounded: a warp that does not see its own copy complete within
// kWaitLimitNs sets GMS_DEV_TIMEOUT in the status word, drains (bounded) what
// it has in flight and returns.
#include "gms_internal.h"

namespace gms {
namespace {

constexpr uint64_t kM1 = 0xBF58476D1CE4E5B9ull;
constexpr uint64_t kM2 = 0x94D049BB133111EBull;
constexpr unsigned long long kDevTimeout = 1ull;     // GMS_DEV_TIMEOUT
constexpr uint64_t kWaitLimitNs = 2000000000ull;     // 2 s per wait
constexpr uint32_t kFull = 0xffffffffu;

struct alignas(16) StageMeta {  // written by lane 0 when a block is issued, read by the warp when it lands
    uint64_t dst;       // destination address of this block
    uint32_t m;         // bytes of this block (1..4096)
    uint32_t slot_last; // bits 0..7: index of the block in its chunk; bit 8: last block of the chunk
    uint32_t gblock0;   // digest slot of the chunk's first block
    uint32_t tblock0;   // tensor-relative index of the chunk's first block
    uint32_t tensor;    // accumulator slot
    uint32_t pad;
};
static_assert(sizeof(StageMeta) == 32, "StageMeta is 32 bytes");

struct Item {  // one chunk as the pipeline sees it
    const uint8_t *src;
    uint8_t *dst;
    uint32_t nbytes, tensor, gblock0, tblock0;
};

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}
__device__ __forceinline__ uint64_t global_timer_ns()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Wait for a phase of one of the warp's own barriers; false after kWaitLimitNs.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity)
{
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_timer_ns();
    for (uint32_t outer = 0; outer < (1u << 24); ++outer) {
#pragma unroll 1
        for (int i = 0; i < 32; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (global_timer_ns() - t0 > kWaitLimitNs) return false;
    }
    return false;
}
// 1-D bulk copy global -> shared (bytes: multiple of 16, both addresses 16-byte aligned).
__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst_smem),
                 "l"(__cvta_generic_to_global(src)), "r"(bytes), "r"(bar)
                 : "memory");
}
// 1-D bulk copy shared -> global, tracked by the thread's bulk async-group.
__device__ __forceinline__ void bulk_store(void *dst, uint32_t src_smem, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(__cvta_generic_to_global(dst)),
                 "r"(src_smem), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read()
{
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// ---------------------------------------------------------------- digest arithmetic
__device__ __forceinline__ uint64_t mix_full(uint64_t z)
{
    z = (z ^ (z >> 30)) * kM1;
    z = (z ^ (z >> 27)) * kM2;
    return z ^ (z >> 31);
}
// mix(w ^ c) without its last xor-shift; cfold = c ^ (c >> 30).
__device__ __forceinline__ uint64_t mix_head(uint64_t w, uint64_t cfold)
{
    uint64_t z = (w ^ (w >> 30) ^ cfold) * kM1;
    z = (z ^ (z >> 27)) * kM2;
    return z;
}
__device__ __forceinline__ uint64_t warp_xor64(uint64_t v)
{
    uint32_t lo = __reduce_xor_sync(kFull, (uint32_t)v);
    uint32_t hi = __reduce_xor_sync(kFull, (uint32_t)(v >> 32));
    return ((uint64_t)hi << 32) | lo;
}

// ---------------------------------------------------------------- chunk providers (warp-uniform)
struct ListProvider {
    const Chunk *chunks;
    uint32_t n_chunks;
    unsigned int *counter;
    const uint8_t *image;  // null: digest in place (source = destination)
    __device__ __forceinline__ bool next(Item &it, uint32_t lane)
    {
        uint32_t idx = 0;
        if (lane == 0) idx = atomicAdd(counter, 1u);
        idx = __shfl_sync(kFull, idx, 0);
        if (idx >= n_chunks) return false;
        const uint4 *p = reinterpret_cast<const uint4 *>(chunks + idx);
        const uint4 a = __ldg(p), b = __ldg(p + 1);
        const uint64_t src_off = ((uint64_t)a.y << 32) | a.x;
        it.dst = reinterpret_cast<uint8_t *>(((uint64_t)a.w << 32) | a.z);
        it.src = image ? image + src_off : it.dst;
        it.nbytes = b.x;
        it.tensor = b.y;
        it.gblock0 = b.z;
        it.tblock0 = b.w;
        return true;
    }
};

struct KvProvider {
    KvArgs a;
    uint64_t unit, stride, total;  // unit = j * n_planes + p
    __device__ __forceinline__ bool next(Item &it, uint32_t lane)
    {
        const uint32_t k = a.block_bytes >> 12;
        while (unit < total) {
            const uint32_t j = (uint32_t)(unit / a.n_planes), p = (uint32_t)(unit % a.n_planes);
            const uint64_t u = unit;
            unit += stride;
            const int32_t id = __ldg(a.ids + j);
            if (id < 0 || (uint32_t)id >= a.n_blocks) {  // skipped: digests 0, counted once per id
                if (a.block_digests && lane < k) a.block_digests[u * k + lane] = 0;
                if (p == 0 && lane == 0) atomicAdd(a.status, 1ull);
                continue;
            }
            it.src = a.image + (uint64_t)p * a.img_plane_stride + (uint64_t)j * a.img_slot_stride;
            it.dst = a.pool_base + (uint64_t)p * a.plane_stride + (uint64_t)id * a.block_stride;
            it.nbytes = a.block_bytes;
            it.tensor = j;
            it.gblock0 = (uint32_t)(u * k);
            it.tblock0 = p * k;
            return true;
        }
        return false;
    }
};

// ---------------------------------------------------------------- the per-warp pipeline
template <int S, bool kStore, class Provider>
__device__ __forceinline__ void run_pipeline(Provider &prov, uint8_t *ring, StageMeta *meta, uint64_t *bars,
                                             uint64_t *block_digests, uint64_t *accum, unsigned long long *status)
{
    constexpr uint32_t LOOK = S - 1;  // blocks in flight ahead of the one being digested
    const uint32_t lane = threadIdx.x & 31u;

    // folded position constants of the 16 words this lane sees in every block:
    // 16-byte load j (0..7) of lane l covers words 64 j + 2 l and 64 j + 2 l + 1.
    uint64_t cfold[16];
#pragma unroll
    for (int j = 0; j < 8; ++j)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const uint64_t c = (uint64_t)(64 * j + 2 * lane + e) * kG;
            cfold[2 * j + e] = c ^ (c >> 30);
        }

    const uint32_t ring_s = smem_u32(ring), bars_s = smem_u32(bars);
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < S; ++s) mbar_init(bars_s + 8u * s, 1u);
        fence_mbar_init();
    }
    __syncwarp();

    Item it{};
    uint32_t it_blocks = 0, it_next = 0;
    bool more = true, failed = false;
    uint32_t issued = 0, consumed = 0;
    uint64_t myD = 0;

    for (;;) {
        // ---------------- issue: keep LOOK blocks ahead
        while (more && issued - consumed < LOOK) {
            if (it_next == it_blocks) {
                more = prov.next(it, lane);
                if (!more) break;
                it_blocks = (it.nbytes + kBlockBytes - 1) >> 12;
                it_next = 0;
            }
            const uint32_t s = issued % S;
            const uint32_t off = it_next << 12;
            const uint32_t m = min(kBlockBytes, it.nbytes - off);
            const uint32_t m16 = m & ~15u;
            uint8_t *stage = ring + s * kBlockBytes;
            // the slot was last read by the store of block issued-S: all but the newest group must have read
            if (kStore && lane == 0) bulk_wait_read<S - LOOK>();
            if (m < kBlockBytes) {
                // short last block of a tensor: zero-fill the slot past the bulk part and move the <16 B tail by hand
                __syncwarp();
                for (uint32_t o = m16 + 16u * lane; o < kBlockBytes; o += 512u)
                    *reinterpret_cast<uint4 *>(stage + o) = make_uint4(0, 0, 0, 0);
                __syncwarp();
                if (lane < (m & 15u)) {
                    const uint8_t v = it.src[off + m16 + lane];
                    stage[m16 + lane] = v;
                    if (kStore) it.dst[off + m16 + lane] = v;
                }
                fence_proxy_async_smem();  // generic writes to a slot that bulk copies will overwrite later
                __syncwarp();
            }
            if (lane == 0) {
                StageMeta md;
                md.dst = reinterpret_cast<uint64_t>(it.dst + off);
                md.m = m;
                md.slot_last = it_next | ((it_next + 1 == it_blocks) ? 256u : 0u);
                md.gblock0 = it.gblock0;
                md.tblock0 = it.tblock0;
                md.tensor = it.tensor;
                md.pad = 0;
                meta[s] = md;
                mbar_arrive_expect_tx(bars_s + 8u * s, m16);
                if (m16) bulk_load(ring_s + s * kBlockBytes, it.src + off, m16, bars_s + 8u * s);
            }
            ++it_next;
            ++issued;
        }
        if (consumed == issued) break;

        // ---------------- consume block `consumed`
        const uint32_t s = consumed % S;
        const bool ok = mbar_wait_bounded(bars_s + 8u * s, (consumed / S) & 1u);
        if (!__all_sync(kFull, ok)) {
            failed = true;
            break;
        }
        __syncwarp();
        const uint4 m0 = *reinterpret_cast<const uint4 *>(&meta[s]);
        const uint4 m1 = *(reinterpret_cast<const uint4 *>(&meta[s]) + 1);
        const uint8_t *stage = ring + s * kBlockBytes;
        if (kStore && lane == 0) {
            const uint32_t m16 = m0.z & ~15u;
            if (m16) bulk_store(reinterpret_cast<void *>(((uint64_t)m0.y << 32) | m0.x), ring_s + s * kBlockBytes, m16);
            bulk_commit();
        }
        uint64_t acc = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint4 v = *reinterpret_cast<const uint4 *>(stage + 512 * j + 16 * lane);
            acc ^= mix_head(((uint64_t)v.y << 32) | v.x, cfold[2 * j]);
            acc ^= mix_head(((uint64_t)v.w << 32) | v.z, cfold[2 * j + 1]);
        }
        acc = warp_xor64(acc);
        const uint64_t D = acc ^ (acc >> 31);
        const uint32_t slot = m0.w & 255u;
        if (lane == slot) myD = D;
        if (m0.w & 256u) {  // chunk complete: block digests leave coalesced, one atomic for the tensor digest
            const uint32_t gblock0 = m1.x, tblock0 = m1.y, tensor = m1.z;
            uint64_t t = 0;
            if (lane <= slot) {
                if (block_digests) block_digests[(uint64_t)gblock0 + lane] = myD;
                t = mix_full(myD ^ ((uint64_t)(tblock0 + lane) * kG));
            }
            t = warp_xor64(t);
            if (lane == 0 && accum) atomicXor(reinterpret_cast<unsigned long long *>(accum + tensor), (unsigned long long)t);
        }
        __syncwarp();  // every lane is done reading the slot before it is refilled
        ++consumed;
    }

    if (failed) {
        if (lane == 0) atomicOr(status, kDevTimeout);
        // bounded drain of what is still in flight into this warp's ring
        for (uint32_t b = consumed; b != issued; ++b) (void)mbar_wait_bounded(bars_s + 8u * (b % S), (b / S) & 1u);
    }
    if (kStore && lane == 0) bulk_wait_all();
}

struct SmemLayout {
    uint8_t *ring;
    StageMeta *meta;
    uint64_t *bars;
};
template <int S>
__device__ __forceinline__ SmemLayout carve(uint8_t *smem)
{
    const uint32_t warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    SmemLayout l;
    l.ring = smem + (size_t)warp * S * kBlockBytes;
    uint8_t *after = smem + (size_t)nwarps * S * kBlockBytes;
    l.meta = reinterpret_cast<StageMeta *>(after) + warp * S;
    l.bars = reinterpret_cast<uint64_t *>(after + (size_t)nwarps * S * sizeof(StageMeta)) + warp * S;
    return l;
}

template <int S, bool kStore>
__global__ void __launch_bounds__(512, 1) gms_stream_kernel(StreamArgs a)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    const SmemLayout l = carve<S>(smem);
    ListProvider prov{a.chunks, a.n_chunks, a.work_counter, kStore ? a.image : nullptr};
    run_pipeline<S, kStore>(prov, l.ring, l.meta, l.bars, a.block_digests, a.tensor_digests, a.status);
}

template <int S>
__global__ void __launch_bounds__(512, 1) gms_kv_stream_kernel(KvArgs a)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    const SmemLayout l = carve<S>(smem);
    const uint32_t nwarps = blockDim.x >> 5;
    KvProvider prov{a, (uint64_t)blockIdx.x * nwarps + (threadIdx.x >> 5), (uint64_t)gridDim.x * nwarps,
                    (uint64_t)a.n_sel * a.n_planes};
    run_pipeline<S, true>(prov, l.ring, l.meta, l.bars, a.block_digests, a.kv_digests, a.status + 1);
}

// Clears the accumulators the streaming kernels XOR / add into.
__global__ void gms_prologue_kernel(uint64_t *accum, uint64_t n_accum, unsigned int *counter, unsigned long long *status,
                                    uint32_t n_status)
{
    const uint64_t i0 = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x, step = (uint64_t)gridDim.x * blockDim.x;
    if (accum)
        for (uint64_t i = i0; i < n_accum; i += step) accum[i] = 0;
    if (i0 == 0 && counter) *counter = 0;
    if (i0 < n_status) status[i0] = 0;
}

uint32_t env_u32(const char *name, uint32_t dflt)
{
    const char *v = getenv(name);
    if (!v || !*v) return dflt;
    char *end = nullptr;
    unsigned long x = strtoul(v, &end, 10);
    return (end && *end == 0 && x > 0 && x < 1024) ? (uint32_t)x : dflt;
}

template <int S>
cudaError_t set_attrs(uint32_t smem)
{
    cudaError_t e;
    if ((e = cudaFuncSetAttribute(gms_stream_kernel<S, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem))) return e;
    if ((e = cudaFuncSetAttribute(gms_stream_kernel<S, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem))) return e;
    return cudaFuncSetAttribute(gms_kv_stream_kernel<S>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
}

constexpr int kMaxDevices = 64;
Geometry g_geom[kMaxDevices];
bool g_geom_ok[kMaxDevices];

cudaError_t prologue(uint64_t *accum, uint64_t n_accum, unsigned int *counter, unsigned long long *status, uint32_t n_status,
                     cudaStream_t s)
{
    const uint32_t threads = 256;
    uint64_t blocks = accum ? (n_accum + threads - 1) / threads : 1;
    if (blocks < 1) blocks = 1;
    if (blocks > 1184) blocks = 1184;
    gms_prologue_kernel<<<(uint32_t)blocks, threads, 0, s>>>(accum, n_accum, counter, status, n_status);
    count_launches(1);
    return cudaGetLastError();
}

template <bool kStore>
cudaError_t launch_stream(const StreamArgs &a, cudaStream_t s)
{
    Geometry g;
    cudaError_t e = get_geometry(&g);
    if (e) return e;
    if ((e = prologue(a.tensor_digests, a.n_tensors, a.work_counter, a.status, 1, s))) return e;
    if (a.n_chunks == 0) return cudaSuccess;
    switch (g.stages) {
    case 3: gms_stream_kernel<3, kStore><<<g.grid, g.warps * 32, g.smem, s>>>(a); break;
    case 6: gms_stream_kernel<6, kStore><<<g.grid, g.warps * 32, g.smem, s>>>(a); break;
    case 8: gms_stream_kernel<8, kStore><<<g.grid, g.warps * 32, g.smem, s>>>(a); break;
    default: gms_stream_kernel<4, kStore><<<g.grid, g.warps * 32, g.smem, s>>>(a); break;
    }
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace

cudaError_t get_geometry(Geometry *out)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    if (!g_geom_ok[dev]) {
        int sms = 0, max_smem = 0;
        if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev))) return e;
        if ((e = cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev))) return e;
        Geometry g;
        // internal tuning hooks (defaults are what the benchmark numbers were taken with)
        g.warps = env_u32("GMS_WARPS", 12);
        g.stages = env_u32("GMS_STAGES", 4);
        const uint32_t per_sm = env_u32("GMS_CTAS_PER_SM", 1);
        if (g.stages != 3 && g.stages != 4 && g.stages != 6 && g.stages != 8) g.stages = 4;
        if (g.warps > 16) g.warps = 16;
        auto need = [&](uint32_t w) { return w * g.stages * (uint32_t)(kBlockBytes + sizeof(StageMeta) + 8); };
        while (g.warps > 1 && need(g.warps) * per_sm > (uint32_t)max_smem) --g.warps;
        g.smem = need(g.warps);
        g.grid = (uint32_t)sms * per_sm;
        switch (g.stages) {
        case 3: e = set_attrs<3>(g.smem); break;
        case 6: e = set_attrs<6>(g.smem); break;
        case 8: e = set_attrs<8>(g.smem); break;
        default: e = set_attrs<4>(g.smem); break;
        }
        if (e) return e;
        g_geom[dev] = g;
        g_geom_ok[dev] = true;
    }
    *out = g_geom[dev];
    return cudaSuccess;
}

cudaError_t launch_restore(const StreamArgs &a, cudaStream_t s) { return launch_stream<true>(a, s); }
cudaError_t launch_digest(const StreamArgs &a, cudaStream_t s) { return launch_stream<false>(a, s); }

cudaError_t launch_kv_restore(const KvArgs &a, cudaStream_t s)
{
    Geometry g;
    cudaError_t e = get_geometry(&g);
    if (e) return e;
    if ((e = prologue(a.kv_digests, a.n_sel, nullptr, a.status, 2, s))) return e;
    if (a.n_sel == 0 || a.n_planes == 0) return cudaSuccess;
    switch (g.stages) {
    case 3: gms_kv_stream_kernel<3><<<g.grid, g.warps * 32, g.smem, s>>>(a); break;
    case 6: gms_kv_stream_kernel<6><<<g.grid, g.warps * 32, g.smem, s>>>(a); break;
    case 8: gms_kv_stream_kernel<8><<<g.grid, g.warps * 32, g.smem, s>>>(a); break;
    default: gms_kv_stream_kernel<4><<<g.grid, g.warps * 32, g.smem, s>>>(a); break;
    }
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace gms
