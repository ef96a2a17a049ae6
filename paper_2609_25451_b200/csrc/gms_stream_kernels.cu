// Persistent streaming kernels of the restore / digest path (sm_100a).
//
// Shape of the work.  A restore is HBM-bound: every payload byte is read once
// and written once, and the digest costs ~17 integer instructions per 8-byte
// word, which fits under the memory time.  Nothing here is a contraction, so
// no tensor cores; what matters is bytes in flight, full-line transactions and
// no per-tensor launches.
//
// Design.  One CTA per SM (9 warps x 4 ring slots for restore / capture, 8 x 6 for the
// KV copies, 16 x 3 for digest-only), and every warp is its own small pipeline with no CTA-wide
// synchronisation at all:
//   * the warp claims a chunk (by default 4 digest blocks = 16 KiB of one tensor,
//     at most 32) from the manifest's work list with one atomicAdd, drawn one
//     chunk ahead of its use so the atomic's latency is never exposed -- no warp
//     ever waits for another.  The copying kernels draw from a single counter:
//     chunks are then started in strict list (= address) order, all bytes in
//     flight lie in a narrow moving window of the image, and HBM rewards that
//     (measured: +3..5 % over round-robin or interleaved counters);
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
#include <algorithm>
#include <mutex>

#include "gms_internal.h"

namespace gms {
namespace {

constexpr uint64_t kM1 = 0xBF58476D1CE4E5B9ull;
constexpr uint64_t kM2 = 0x94D049BB133111EBull;
constexpr unsigned long long kDevTimeout = 1ull;     // GMS_DEV_TIMEOUT
constexpr uint64_t kWaitLimitNs = 2000000000ull;     // 2 s per wait
constexpr uint32_t kFull = 0xffffffffu;

struct Item {  // one chunk as the pipeline sees it
    const uint8_t *src;
    uint8_t *dst;
    uint32_t nbytes, tensor, gblock0, tblock0;
    uint32_t stall;  // self-test only: bytes announced on the first block's barrier that never arrive (else 0)
};

constexpr uint32_t kFifo = 8;  // chunk records in flight between a warp's issue side and its digest side (>= ring slots)

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
// Wait for a phase of one of the warp's own barriers until the global timer passes `deadline`; false if it did.
__device__ __forceinline__ bool mbar_wait_until(uint32_t bar, uint32_t parity, uint64_t deadline)
{
    for (uint32_t outer = 0; outer < (1u << 24); ++outer) {
#pragma unroll 1
        for (int i = 0; i < 32; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (global_timer_ns() > deadline) return false;
    }
    return false;
}
// Wait for a phase of one of the warp's own barriers; false after kWaitLimitNs.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity)
{
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_until(bar, parity, global_timer_ns() + kWaitLimitNs);
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
// The same load with an L2 eviction policy attached (used by the digest-only kernels, see kL2KeepBytes).
__device__ __forceinline__ void bulk_load_hint(uint32_t dst_smem, const void *src, uint32_t bytes, uint32_t bar, uint64_t policy)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                 ::"r"(dst_smem), "l"(__cvta_generic_to_global(src)), "r"(bytes), "r"(bar), "l"(policy)
                 : "memory");
}
__device__ __forceinline__ uint64_t l2_policy_evict_first()
{
    uint64_t p;
    asm("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_last()
{
    uint64_t p;
    asm("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ void store_u64_hint(uint64_t *p, uint64_t v, uint64_t policy)
{
    asm volatile("st.global.L2::cache_hint.u64 [%0], %1, %2;" ::"l"(p), "l"(v), "l"(policy) : "memory");
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
// Three-input XOR in one LOP3.
__device__ __forceinline__ uint32_t xor3(uint32_t a, uint32_t b, uint32_t c)
{
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0x96;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
// Low 64 bits of (th:tl) * (Mh:Ml): one widening multiply and two multiply-adds.
__device__ __forceinline__ void mul64_lo(uint32_t tl, uint32_t th, uint32_t Ml, uint32_t Mh, uint32_t &pl, uint32_t &ph)
{
    asm("{\n\t.reg .u64 p;\n\tmul.wide.u32 p, %2, %3;\n\tmov.b64 {%0, %1}, p;\n\t}" : "=r"(pl), "=r"(ph) : "r"(tl), "r"(Ml));
    asm("mad.lo.u32 %0, %1, %2, %0;" : "+r"(ph) : "r"(tl), "r"(Mh));
    asm("mad.lo.u32 %0, %1, %2, %0;" : "+r"(ph) : "r"(th), "r"(Ml));
}
// mix(w ^ c) without its last xor-shift, on 32-bit halves; (cl, ch) = c ^ (c >> 30).
// Spelled out so that a word costs exactly 2 widening multiplies, 4 multiply-adds, 4 shifts and 4 LOP3 (plus one
// LOP3 per word for the running XOR): the compiler's lowering of the plain 64-bit form executes 8.5 multiply-pipe
// and 11.6 ALU instructions per word (register moves, two-input XORs), this one 6.6 and 9.5 -- measured on a
// block already in shared memory: 11.4 TB/s of payload against 9.8 at 1965 MHz.  Spelling the shifts as
// multiplies by powers of two (to move them to the multiply pipe) was measured too and is slower (7.0-10.4 TB/s):
// the widening and high-half multiplies cost the pipe twice what a low-half multiply-add does.
__device__ __forceinline__ void mix_head32(uint32_t lo, uint32_t hi, uint32_t cl, uint32_t ch, uint32_t &ql, uint32_t &qh)
{
    constexpr uint32_t M1l = (uint32_t)kM1, M1h = (uint32_t)(kM1 >> 32), M2l = (uint32_t)kM2, M2h = (uint32_t)(kM2 >> 32);
    const uint32_t tl = xor3(lo, __funnelshift_r(lo, hi, 30), cl), th = xor3(hi, hi >> 30, ch);
    uint32_t zl, zh;
    mul64_lo(tl, th, M1l, M1h, zl, zh);
    const uint32_t ul = zl ^ __funnelshift_r(zl, zh, 27), uh = zh ^ (zh >> 27);
    mul64_lo(ul, uh, M2l, M2h, ql, qh);
}
// The whole mix, for the tensor digest (once per block digest).
__device__ __forceinline__ uint64_t mix_full32(uint64_t z)
{
    uint32_t ql, qh;
    mix_head32((uint32_t)z, (uint32_t)(z >> 32), 0u, 0u, ql, qh);
    const uint64_t y = ((uint64_t)qh << 32) | ql;
    return y ^ (y >> 31);
}
__device__ __forceinline__ uint64_t warp_xor64(uint64_t v)
{
    uint32_t lo = __reduce_xor_sync(kFull, (uint32_t)v);
    uint32_t hi = __reduce_xor_sync(kFull, (uint32_t)(v >> 32));
    return ((uint64_t)hi << 32) | lo;
}

// ---------------------------------------------------------------- chunk providers (warp-uniform)
// Both providers run one step ahead: the claim (an atomic) and the descriptor load for the chunk
// after next are issued when a chunk is handed out and consumed a whole chunk later, so their
// latency never sits between two blocks of a warp's pipeline.
struct ListProvider {
    const Chunk *chunks;
    uint32_t n_chunks;
    unsigned int *counters;  // n_counters work counters, kCounterStride words apart
    uint32_t n_counters;
    const uint8_t *image;    // null: digest in place (source = destination)
    bool capture;            // copy allocation -> image instead of image -> allocation
    uint32_t home;           // the counter this warp is drawing from
    uint32_t exhausted;      // counters found empty so far
    uint32_t raw_next;       // lane 0: ticket drawn from counter `home` one step ahead
    uint32_t group;          // consecutive chunks bought by one ticket
    uint32_t grp_left, grp_idx;
    uint4 da, db;            // buffered descriptor
    uint32_t buffered;       // its index in the list
    uint32_t stall_chunk;    // self-test: the chunk whose first wait is made to run out (0xffffffff: none)
    bool have;

    __device__ __forceinline__ void load(uint32_t idx)
    {
        const uint4 *p = reinterpret_cast<const uint4 *>(chunks + idx);
        da = __ldg(p);
        db = __ldg(p + 1);
        buffered = idx;
    }
    __device__ __forceinline__ void draw(uint32_t lane)
    {
        if (lane == 0) raw_next = atomicAdd(counters + home * kCounterStride, 1u);
    }
    // Counter c hands out chunk runs c, c + n_counters, c + 2 n_counters, ... (a run = `group` consecutive
    // chunks); warps are spread over the counters, so the chunks in flight stay a compact moving front of the
    // work list while no single address takes all the atomics.  A warp whose counter has run dry moves on to
    // the next one (that is the load balancing).  The ticket used here was drawn one step earlier; the next one
    // is drawn now and read a chunk later.
    __device__ __forceinline__ bool advance(uint32_t lane, uint32_t &idx_out)
    {
        if (grp_left) {  // still inside the run of `group` consecutive chunks the last ticket bought
            --grp_left;
            if (++grp_idx < n_chunks) {
                idx_out = grp_idx;
                return true;
            }
            grp_left = 0;  // the run ran off the end of the list: go and draw elsewhere
        }
        for (;;) {
            const uint32_t t = __shfl_sync(kFull, raw_next, 0);
            const uint64_t idx = ((uint64_t)t * n_counters + home) * group;
            if (idx < n_chunks) {
                draw(lane);
                idx_out = grp_idx = (uint32_t)idx;
                grp_left = group - 1;
                return true;
            }
            if (++exhausted >= n_counters) return false;
            home = home + 1 == n_counters ? 0 : home + 1;
            draw(lane);
        }
    }
    __device__ __forceinline__ void init(uint32_t lane)
    {
        home = (blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)) % n_counters;
        exhausted = 0;
        raw_next = 0;
        grp_left = 0;
        grp_idx = 0;
        draw(lane);
        uint32_t idx;
        have = advance(lane, idx);
        if (have) load(idx);
    }
    __device__ __forceinline__ bool next(Item &it, uint32_t lane)
    {
        if (!have) return false;
        const uint64_t src_off = ((uint64_t)da.y << 32) | da.x;
        it.dst = reinterpret_cast<uint8_t *>(((uint64_t)da.w << 32) | da.z);
        it.src = image ? image + src_off : it.dst;
        if (capture) {  // gather: the allocation is the source, the packed image the destination
            const uint8_t *alloc = it.dst;
            it.dst = const_cast<uint8_t *>(it.src);
            it.src = alloc;
        }
        it.nbytes = db.x;
        it.tensor = db.y;
        it.gblock0 = db.z;
        it.tblock0 = db.w;
        it.stall = buffered == stall_chunk ? 16u : 0u;
        uint32_t idx;
        have = advance(lane, idx);
        if (have) load(idx);
        return true;
    }
};

// Units are (plane p, selected slot j).  The copying calls walk them plane-major, so that consecutive
// units read (or write) consecutive 32 KiB runs of the packed image.  The digest-only call has no image
// and walks them slot-major instead: consecutive units then fill consecutive digest slots (the layout
// is [j][p][block]), whole lines at a time, where plane-major leaves 64-byte pieces 4 KiB apart
// (measured on the 60 GB pool: 0.855 against 0.870 ms).  Units are claimed in order from one counter
// (kept in the caller's status array), one step ahead like the list provider, so the reads in flight
// form a compact moving front of the image.
struct KvProvider {
    KvArgs a;
    unsigned int *counter;
    uint32_t total;     // n_planes * n_sel
    uint32_t u_next;    // unit handed out next (already claimed)
    int32_t id_next;    // its pool block id (already loaded)
    uint32_t raw_next;  // lane 0: ticket for the unit after that

    __device__ __forceinline__ void step(uint32_t lane)
    {
        u_next = __shfl_sync(kFull, raw_next, 0);
        if (lane == 0) raw_next = atomicAdd(counter, 1u);
        if (u_next < total) id_next = __ldg(a.ids + (a.digest_only ? u_next / a.n_planes : u_next % a.n_sel));
    }
    __device__ __forceinline__ void init(uint32_t lane)
    {
        raw_next = 0;
        id_next = 0;
        if (lane == 0) raw_next = atomicAdd(counter, 1u);
        step(lane);
    }
    __device__ __forceinline__ bool next(Item &it, uint32_t lane)
    {
        const uint32_t k = a.block_bytes >> 12;
        while (u_next < total) {
            const uint32_t p = a.digest_only ? u_next % a.n_planes : u_next / a.n_sel;
            const uint32_t j = a.digest_only ? u_next / a.n_planes : u_next % a.n_sel;
            const int32_t id = id_next;
            step(lane);
            const uint32_t slot0 = (j * a.n_planes + p) * k;  // digest slots are laid out [j][p][block]
            if (id < 0 || (uint32_t)id >= a.n_blocks) {       // skipped: digests 0, counted once per id
                if (a.block_digests && lane < k) a.block_digests[(uint64_t)slot0 + lane] = 0;
                if (p == 0 && lane == 0) atomicAdd(a.status, 1ull);
                continue;
            }
            const uint32_t img_slot = a.by_id ? (uint32_t)id : j;  // pool-shaped image: slot = block id
            uint8_t *img = const_cast<uint8_t *>(a.image) + (uint64_t)p * a.img_plane_stride + (uint64_t)img_slot * a.img_slot_stride;
            uint8_t *blk = a.pool_base + (uint64_t)p * a.plane_stride + (uint64_t)id * a.block_stride;
            it.src = (a.capture || a.digest_only) ? blk : img;
            it.dst = a.capture ? img : blk;  // unused when digesting in place
            it.nbytes = a.block_bytes;
            it.tensor = j;
            it.gblock0 = slot0;
            it.tblock0 = p * k;
            it.stall = 0;
            return true;
        }
        return false;
    }
};

// ---------------------------------------------------------------- the per-warp pipeline
// `expected` / `seg_count` (both null, or both set): the fused compare.  At the end of a chunk every lane that holds
// a block digest checks it against the recorded one and, if they differ, bumps the counter of the 2048-slot
// segment the block lies in -- the first pass of the ordered compaction in gms_verify_kernels.cu, done here
// while the digest is still in a register, so that gms_digest_verify / gms_restore_verify only run scan + emit.
template <int S, bool kStore, class Provider>
__device__ __forceinline__ void run_pipeline(Provider &prov, uint8_t *ring, uint4 *fifo, uint64_t *bars, uint64_t *block_digests,
                                             uint64_t *accum, unsigned long long *status, const uint64_t *expected,
                                             uint32_t *seg_count, bool l2_keep)
{
    static_assert(S <= (int)kFifo, "the chunk fifo must cover the ring");
    constexpr uint32_t LOOK = S - 1;  // blocks in flight ahead of the one being digested
    const uint32_t lane = threadIdx.x & 31u;

    // folded position constants of the 16 words this lane sees in every block:
    // 16-byte load j (0..7) of lane l covers words 64 j + 2 l and 64 j + 2 l + 1.
    uint32_t cl[16], ch[16];
#pragma unroll
    for (int j = 0; j < 8; ++j)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const uint64_t c = (uint64_t)(64 * j + 2 * lane + e) * kG, f = c ^ (c >> 30);
            cl[2 * j + e] = (uint32_t)f;
            ch[2 * j + e] = (uint32_t)(f >> 32);
        }

    const uint32_t ring_s = smem_u32(ring), bars_s = smem_u32(bars);
    // digest-only kernels with a small output: payload loads evict-first, digest stores evict-last (see kL2KeepBytes)
    const bool keep = !kStore && l2_keep;
    const uint64_t pol_first = l2_policy_evict_first(), pol_last = l2_policy_evict_last();
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < S; ++s) mbar_init(bars_s + 8u * s, 1u);
        fence_mbar_init();
    }
    __syncwarp();
    // Everything above touched registers and this warp's own shared memory only, so it ran while the grid before
    // this one (the prologue that clears counters and accumulators, or whatever the caller enqueued) was still
    // running.  From here on global memory is read and written: wait for that grid's writes.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    prov.init(lane);

    // issue-side cursor (the chunk being fetched) and digest-side cursor (the chunk being consumed);
    // chunk records travel from one to the other through a small per-warp fifo in shared memory
    Item it{};
    uint32_t it_blocks = 0, it_full = 0, it_next = 0, chunks_in = 0, stall_extra = 0;
    uint64_t c_dst = 0;
    uint32_t c_nbytes = 0, c_tensor = 0, c_gblock0 = 0, c_tblock0 = 0, c_blocks = 0, c_next = 0, chunks_out = 0;
    bool more = true, failed = false;
    uint32_t issued = 0, consumed = 0;
    uint32_t is = 0;               // ring slot of the next block to issue   (issued % S)
    uint32_t cs = 0, cparity = 0;  // ring slot and barrier phase of the next block to digest
    uint32_t my_lo = 0, my_hi = 0;
    uint64_t want = 0;  // fused compare: the recorded digest of the block whose digest this lane holds
    // share of a tensor digest gathered over consecutive chunks of the same tensor: one atomic per run, not per chunk
    uint32_t run_tensor = 0xffffffffu;
    uint64_t run_val = 0;

    // ---------------- issue the next block of the work list (false: the list is exhausted)
    auto issue_one = [&]() -> bool {
        {
            if (it_next == it_blocks) {
                more = prov.next(it, lane);
                if (!more) return false;
                it_blocks = (it.nbytes + kBlockBytes - 1) >> 12;
                it_full = it.nbytes >> 12;  // whole blocks: nothing to pad, no hand-moved tail
                stall_extra = it.stall;     // self-test only: announced on the chunk's first barrier, never sent
                it_next = 0;
                if (lane == 0) {
                    const uint64_t d = reinterpret_cast<uint64_t>(it.dst);
                    fifo[2 * (chunks_in % kFifo)] = make_uint4((uint32_t)d, (uint32_t)(d >> 32), it.nbytes, it.tensor);
                    fifo[2 * (chunks_in % kFifo) + 1] = make_uint4(it.gblock0, it.tblock0, 0u, 0u);
                }
                ++chunks_in;
            }
            const uint32_t s = is;
            is = (is + 1 == S) ? 0 : is + 1;
            const uint32_t off = it_next << 12;
            // the slot was last read by the store of block issued-S: all but the newest group must have read
            if (kStore && lane == 0) bulk_wait_read<S - LOOK>();
            uint32_t m16 = kBlockBytes;
            if (it_next >= it_full) {
                // short last block of a tensor: zero-fill the slot past the bulk part and move the <16 B tail by hand
                const uint32_t m = it.nbytes - off;
                m16 = m & ~15u;
                uint8_t *stage = ring + s * kBlockBytes;
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
                mbar_arrive_expect_tx(bars_s + 8u * s, m16 + stall_extra);
                if (m16) {
                    if (keep)
                        bulk_load_hint(ring_s + s * kBlockBytes, it.src + off, m16, bars_s + 8u * s, pol_first);
                    else
                        bulk_load(ring_s + s * kBlockBytes, it.src + off, m16, bars_s + 8u * s);
                }
            }
            stall_extra = 0;
            ++it_next;
            ++issued;
        }
        return true;
    };
    // LOOK blocks go out first; after that every digested block is followed by one more issue, so the warp always
    // has LOOK blocks in flight or in work
    for (uint32_t k = 0; k < LOOK; ++k)
        if (!issue_one()) break;
    while (consumed != issued) {
        // ---------------- digest block `consumed`
        const uint32_t s = cs;
        const bool ok = mbar_wait_bounded(bars_s + 8u * s, cparity);
        if (++cs == S) cs = 0, cparity ^= 1u;
        if (!__all_sync(kFull, ok)) {
            failed = true;
            break;
        }
        __syncwarp();
        if (c_next == c_blocks) {  // next chunk record
            const uint4 r0 = fifo[2 * (chunks_out % kFifo)], r1 = fifo[2 * (chunks_out % kFifo) + 1];
            ++chunks_out;
            c_dst = ((uint64_t)r0.y << 32) | r0.x;
            c_nbytes = r0.z;
            c_tensor = r0.w;
            c_gblock0 = r1.x;
            c_tblock0 = r1.y;
            c_blocks = (c_nbytes + kBlockBytes - 1) >> 12;
            c_next = 0;
            // fused compare: the recorded digests of this chunk's blocks are fetched now and used at its end, so that
            // their latency lies under the chunk's digest work instead of behind it
            if (expected && lane < c_blocks) want = __ldg(expected + c_gblock0 + lane);
        }
        const uint8_t *stage = ring + s * kBlockBytes;
        if (kStore && lane == 0) {
            const uint32_t off = c_next << 12;
            const uint32_t m16 = min(kBlockBytes, c_nbytes - off) & ~15u;
            if (m16) bulk_store(reinterpret_cast<void *>(c_dst + off), ring_s + s * kBlockBytes, m16);
            bulk_commit();
        }
        uint32_t al = 0, ah = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint4 v = *reinterpret_cast<const uint4 *>(stage + 512 * j + 16 * lane);
            uint32_t pl, ph, ql, qh;
            mix_head32(v.x, v.y, cl[2 * j], ch[2 * j], pl, ph);
            mix_head32(v.z, v.w, cl[2 * j + 1], ch[2 * j + 1], ql, qh);
            al = xor3(al, pl, ql);
            ah = xor3(ah, ph, qh);
        }
        al = __reduce_xor_sync(kFull, al);
        ah = __reduce_xor_sync(kFull, ah);
        if (lane == c_next) my_lo = al, my_hi = ah;  // the block's XOR before the last xor-shift, which waits for the chunk's end
        ++c_next;
        if (c_next == c_blocks) {  // chunk complete: block digests leave coalesced, one atomic for the tensor digest
            uint64_t t = 0;
            if (lane < c_blocks) {
                const uint64_t raw = ((uint64_t)my_hi << 32) | my_lo, myD = raw ^ (raw >> 31);
                if (block_digests) {
                    if (keep)
                        store_u64_hint(block_digests + (uint64_t)c_gblock0 + lane, myD, pol_last);
                    else
                        block_digests[(uint64_t)c_gblock0 + lane] = myD;
                }
                if (expected && want != myD) atomicAdd(seg_count + ((c_gblock0 + lane) >> kVerifySegShift), 1u);
                t = mix_full32(myD ^ ((uint64_t)(c_tblock0 + lane) * kG));
            }
            t = warp_xor64(t);
            if (c_tensor != run_tensor) {
                if (run_tensor != 0xffffffffu && lane == 0 && accum)
                    atomicXor(reinterpret_cast<unsigned long long *>(accum + run_tensor), (unsigned long long)run_val);
                run_tensor = c_tensor;
                run_val = 0;
            }
            run_val ^= t;
        }
        __syncwarp();  // every lane is done reading the slot before it is refilled
        ++consumed;
        if (more) issue_one();
    }

    if (run_tensor != 0xffffffffu && lane == 0 && accum)
        atomicXor(reinterpret_cast<unsigned long long *>(accum + run_tensor), (unsigned long long)run_val);
    if (failed) {
        if (lane == 0) atomicOr(status, kDevTimeout);
        // drain what is still in flight into this warp's ring, all of it against one more wait limit
        const uint64_t deadline = global_timer_ns() + kWaitLimitNs;
        for (uint32_t b = consumed; b != issued; ++b) (void)mbar_wait_until(bars_s + 8u * (b % S), (b / S) & 1u, deadline);
    }
    if (kStore && lane == 0) bulk_wait_all();
}

struct SmemLayout {
    uint8_t *ring;
    uint4 *fifo;
    uint64_t *bars;
};
constexpr uint32_t kWarpSmemExtra = kFifo * 32 + 8 * 8;  // fifo + up to 8 barriers
template <int S>
__device__ __forceinline__ SmemLayout carve(uint8_t *smem)
{
    const uint32_t warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    SmemLayout l;
    l.ring = smem + (size_t)warp * S * kBlockBytes;
    uint8_t *extra = smem + (size_t)nwarps * S * kBlockBytes + (size_t)warp * kWarpSmemExtra;
    l.fifo = reinterpret_cast<uint4 *>(extra);
    l.bars = reinterpret_cast<uint64_t *>(extra + kFifo * 32);
    return l;
}

// 16 warps is the most the digest-only shape can use: a seventeenth would put five warps on one of the SM's four
// register files and force the kernel from 110 down to 96 registers, which measured slower (2.42-2.47 ms against
// 2.40 ms for the 8B manifest).
template <int S, bool kStore>
__global__ void __launch_bounds__(512, 1) gms_stream_kernel(StreamArgs a)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    const SmemLayout l = carve<S>(smem);
    ListProvider prov;
    prov.chunks = a.chunks;
    prov.n_chunks = a.n_chunks;
    prov.counters = a.work_counters;
    prov.n_counters = a.n_counters;
    prov.group = a.group;
    prov.image = kStore ? a.image : nullptr;
    prov.capture = kStore && a.capture;
    prov.stall_chunk = a.stall_chunk;
    // whatever follows on the stream may be scheduled now; every kernel of this library waits (griddepcontrol.wait)
    // for the grid before it to finish before it touches global memory
    asm volatile("griddepcontrol.launch_dependents;");
    run_pipeline<S, kStore>(prov, l.ring, l.fifo, l.bars, a.block_digests, a.tensor_digests, a.status, a.expected,
                            a.seg_count, a.l2_keep != 0);
}

template <int S, bool kStore>
__global__ void __launch_bounds__(512, 1) gms_kv_stream_kernel(KvArgs a)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    const SmemLayout l = carve<S>(smem);
    KvProvider prov;
    prov.a = a;
    prov.counter = reinterpret_cast<unsigned int *>(a.status + 2);
    prov.total = a.n_sel * a.n_planes;
    asm volatile("griddepcontrol.launch_dependents;");
    run_pipeline<S, kStore>(prov, l.ring, l.fifo, l.bars, a.block_digests, a.kv_digests, a.status + 1, nullptr, nullptr,
                            a.l2_keep != 0);
}

// Clears the accumulators the streaming kernels XOR / add into (and, for the fused compare, the per-segment
// mismatch counters).
__global__ void gms_prologue_kernel(uint64_t *accum, uint64_t n_accum, unsigned int *counters, uint32_t n_counters,
                                    unsigned long long *status, uint32_t n_status, uint32_t *seg_count, uint32_t n_segments)
{
    // let the streaming kernel that follows be scheduled now: it sets itself up (constants, barriers) while this
    // grid runs, and waits (griddepcontrol.wait) for this grid's writes before it touches a counter
    asm volatile("griddepcontrol.launch_dependents;");
    // this grid may itself have been scheduled early, behind a kernel of this library that is still using the
    // counters: wait for it before clearing anything
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const uint64_t i0 = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x, step = (uint64_t)gridDim.x * blockDim.x;
    if (accum)
        for (uint64_t i = i0; i < n_accum; i += step) accum[i] = 0;
    if (seg_count)
        for (uint64_t i = i0; i < n_segments; i += step) seg_count[i] = 0;
    if (i0 < n_counters) counters[i0 * kCounterStride] = 0;
    if (i0 < n_status) status[i0] = 0;
}

// Tuning and test hooks are honoured only when GMS_TUNING_HOOKS=1 is set as well.
const char *hook(const char *name)
{
    const char *on = getenv("GMS_TUNING_HOOKS");
    return on && atoi(on) == 1 ? getenv(name) : nullptr;
}

// "w,s,c" from the environment (tuning hook), else the defaults
void env_geom(const char *name, uint32_t &w, uint32_t &s, uint32_t &c)
{
    const char *v = hook(name);
    unsigned a = 0, b = 0, d = 0;
    if (v && sscanf(v, "%u,%u,%u", &a, &b, &d) == 3 && a >= 1 && a <= 16 && (b == 3 || b == 4 || b == 6 || b == 8) && d >= 1 && d <= 4) {
        w = a;
        s = b;
        c = d;
    }
}

template <int S>
cudaError_t set_attrs(Kind kind, uint32_t smem)
{
    const void *f = kind == kRestore ? (const void *)gms_stream_kernel<S, true>
                    : kind == kDigest ? (const void *)gms_stream_kernel<S, false>
                    : kind == kKv     ? (const void *)gms_kv_stream_kernel<S, true>
                                      : (const void *)gms_kv_stream_kernel<S, false>;
    return cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
}

constexpr int kMaxDevices = 64;
Geometry g_geom[kMaxDevices][kKinds];
bool g_geom_ok[kMaxDevices][kKinds];

// Launch attribute shared by every kernel of the library: the grid may be scheduled while its predecessor on the
// stream still runs (programmatic dependent launch); each kernel waits for the predecessor itself.
cudaLaunchConfig_t pdl_config(dim3 grid, dim3 block, size_t smem, cudaStream_t s, cudaLaunchAttribute *attr)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cfg;
}

cudaError_t prologue(uint64_t *accum, uint64_t n_accum, unsigned int *counters, uint32_t n_counters, unsigned long long *status,
                     uint32_t n_status, uint32_t *seg_count, uint32_t n_segments, cudaStream_t s)
{
    const uint32_t threads = 256;
    uint64_t blocks = std::max<uint64_t>(accum ? (n_accum + threads - 1) / threads : 1, seg_count ? (n_segments + threads - 1) / threads : 1);
    if (blocks < 1) blocks = 1;
    if (blocks > 1184) blocks = 1184;
    cudaLaunchAttribute attr[1];
    cudaLaunchConfig_t cfg = pdl_config(dim3((uint32_t)blocks), dim3(threads), 0, s, attr);
    count_launches(1);
    return cudaLaunchKernelEx(&cfg, gms_prologue_kernel, accum, n_accum, counters, n_counters, status, n_status, seg_count, n_segments);
}

// A streaming kernel is always enqueued right behind its prologue.  Programmatic dependent launch lets the
// hardware schedule it while the prologue still runs (the kernel itself waits before its first claim), which
// hides one launch gap -- all of the difference for manifests of a few megabytes.
template <class Args>
cudaError_t launch_after_prologue(void (*kernel)(Args), const Geometry &g, cudaStream_t s, const Args &args)
{
    cudaLaunchAttribute attr[1];
    cudaLaunchConfig_t cfg = pdl_config(dim3(g.grid), dim3(g.warps * 32), g.smem, s, attr);
    return cudaLaunchKernelEx(&cfg, kernel, args);
}

template <bool kStore>
cudaError_t launch_stream(const StreamArgs &a, cudaStream_t s)
{
    Geometry g;
    cudaError_t e = get_geometry(kStore ? kRestore : kDigest, &g);
    if (e) return e;
    // a windowed restore keeps the tensor-digest accumulators and the status word of its earlier windows
    if ((e = prologue(a.keep_accum ? nullptr : a.tensor_digests, a.n_tensors, a.work_counters, g.counters, a.status,
                      a.keep_accum ? 0 : 1, a.keep_accum ? nullptr : a.seg_count, a.n_segments, s)))
        return e;
    if (a.n_chunks == 0) return cudaSuccess;
    StreamArgs b = a;
    b.n_counters = g.counters;
    // a claim buys a run of chunks only while there are runs enough for every warp
    b.group = (uint32_t)std::min<uint64_t>(g.group, std::max<uint64_t>(1, a.n_chunks / (4ull * g.grid * g.warps)));
    if (b.group == 1 && a.n_chunks < 4ull * g.grid * g.warps) b.n_counters = std::min<uint32_t>(b.n_counters, 2);
    switch (g.stages) {
    case 3: e = launch_after_prologue(gms_stream_kernel<3, kStore>, g, s, b); break;
    case 6: e = launch_after_prologue(gms_stream_kernel<6, kStore>, g, s, b); break;
    case 8: e = launch_after_prologue(gms_stream_kernel<8, kStore>, g, s, b); break;
    default: e = launch_after_prologue(gms_stream_kernel<4, kStore>, g, s, b); break;
    }
    count_launches(1);
    return e;
}

}  // namespace

cudaError_t get_geometry(Kind kind, Geometry *out)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    static std::mutex mu;  // the table is filled once per (device, kernel); callers may come from several threads
    std::lock_guard<std::mutex> lock(mu);
    if (!g_geom_ok[dev][kind]) {
        int sms = 0, max_smem = 0;
        if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev))) return e;
        if ((e = cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev))) return e;
        Geometry g;
        uint32_t per_sm = 1;
        // defaults are what the benchmark numbers were taken with
        if (kind == kDigest || kind == kKvDigest) {
            g.warps = 16, g.stages = 3;
            env_geom("GMS_GEOM_DIGEST", g.warps, g.stages, per_sm);
        } else if (kind == kRestore) {
            // 9 x 4: as fast as 8 x 6 at full clocks (4.70 vs 4.68 ms on the 8B manifest) and 2-3 % faster when a long
            // run has the SM clock power-capped (4.71 vs 4.78-4.90 ms): the ninth warp covers the longer per-block latency
            g.warps = 9, g.stages = 4;
            env_geom("GMS_GEOM_RESTORE", g.warps, g.stages, per_sm);
        } else {
            g.warps = 8, g.stages = 6;
            env_geom("GMS_GEOM_KV", g.warps, g.stages, per_sm);
        }
        auto need = [&](uint32_t w) { return w * (g.stages * kBlockBytes + kWarpSmemExtra); };
        while (g.warps > 1 && (need(g.warps) + 1024) * per_sm > (uint32_t)max_smem) --g.warps;
        g.smem = need(g.warps);
        g.grid = (uint32_t)sms * per_sm;
        // claims: the restore kernels draw single chunks from one counter (strict list order keeps the bytes in
        // flight a compact front, which HBM rewards); the digest kernel claims twice as often per second, so it
        // spreads its claims over two counters (one ticket buys one 32 KiB chunk of its own, longer-cut list:
        // measured 2.24-2.26 ms on the 8B manifest against 2.26-2.29 with 1, 8 or 16 counters and 2.38 with
        // two chunks per ticket)
        g.counters = kind == kDigest ? 2 : 1;
        g.group = 1;
        if (const char *v = hook(kind == kDigest ? "GMS_CLAIM_DIGEST" : "GMS_CLAIM_RESTORE")) {
            unsigned x = 0, y = 0;
            if (sscanf(v, "%u,%u", &x, &y) == 2 && x >= 1 && x <= kMaxCounters && y >= 1 && y <= 64) g.counters = x, g.group = y;
        }
        switch (g.stages) {
        case 3: e = set_attrs<3>(kind, g.smem); break;
        case 6: e = set_attrs<6>(kind, g.smem); break;
        case 8: e = set_attrs<8>(kind, g.smem); break;
        default: e = set_attrs<4>(kind, g.smem); break;
        }
        if (e) return e;
        g_geom[dev][kind] = g;
        g_geom_ok[dev][kind] = true;
    }
    *out = g_geom[dev][kind];
    return cudaSuccess;
}

cudaError_t launch_restore(const StreamArgs &a, cudaStream_t s) { return launch_stream<true>(a, s); }
cudaError_t launch_digest(const StreamArgs &a, cudaStream_t s) { return launch_stream<false>(a, s); }

cudaError_t launch_kv_restore(const KvArgs &a, cudaStream_t s)
{
    Geometry g;
    cudaError_t e = get_geometry(a.digest_only ? kKvDigest : kKv, &g);
    if (e) return e;
    if ((e = prologue(a.kv_digests, a.n_sel, nullptr, 0, a.status, 4, nullptr, 0, s))) return e;
    if (a.n_sel == 0 || a.n_planes == 0) return cudaSuccess;
    const KvArgs &b = a;
    if (a.digest_only) {
        switch (g.stages) {
        case 3: e = launch_after_prologue(gms_kv_stream_kernel<3, false>, g, s, b); break;
        case 6: e = launch_after_prologue(gms_kv_stream_kernel<6, false>, g, s, b); break;
        case 8: e = launch_after_prologue(gms_kv_stream_kernel<8, false>, g, s, b); break;
        default: e = launch_after_prologue(gms_kv_stream_kernel<4, false>, g, s, b); break;
        }
    } else {
        switch (g.stages) {
        case 3: e = launch_after_prologue(gms_kv_stream_kernel<3, true>, g, s, b); break;
        case 6: e = launch_after_prologue(gms_kv_stream_kernel<6, true>, g, s, b); break;
        case 8: e = launch_after_prologue(gms_kv_stream_kernel<8, true>, g, s, b); break;
        default: e = launch_after_prologue(gms_kv_stream_kernel<4, true>, g, s, b); break;
        }
    }
    count_launches(1);
    return e;
}

}  // namespace gms
