// Host side of the C ABI declared in include/gms.h: validation of the layout
// record, construction of the persistent kernels' work list, and the entry
// points that enqueue the kernels.  There is no CPU implementation of the data
// path here: every entry point either launches the CUDA kernels or fails.
#include <algorithm>
#include <atomic>
#include <cstdlib>
#include <cstring>
#include <map>
#include <mutex>
#include <new>
#include <numeric>
#include <string>
#include <vector>

#include "../../include/gms.h"
#include "gms_internal.h"

using gms::Chunk;

struct gms_manifest {
    std::vector<gms_entry> entries;
    std::vector<uint64_t> block_base;  // n + 1 prefix sums of per-tensor block counts
    // The two work lists live on the device, where they are also written (gms_build_kernels.cu).  Host copies are made
    // only when something asks for them: the introspection calls, the window plan of a piecewise restore, a check.
    uint32_t chunk_blocks = 4, digest_chunk_blocks = 8;  // 4 KiB blocks per chunk of the copy list / the digest list
    uint64_t n_chunks = 0, n_digest_chunks = 0;
    mutable std::vector<Chunk> chunks;         // work list of the copying kernels (restore, capture)
    mutable std::vector<Chunk> digest_chunks;  // work list of the digest-only kernel: the same tensors cut into longer runs
    mutable bool host_lists = false;
    uint64_t image_bytes = 0, payload = 0, n_blocks = 0;
    bool host_only = false;
    bool selftest_stall = false;  // GMS_BUILD_SELFTEST_STALL
    bool sources_disjoint = true;  // image ranges pairwise disjoint (needed by gms_capture only)
    int device = -1;
    // device tables (one allocation) and the recorded digests (allocated on first use)
    uint8_t *d_tables = nullptr;
    Chunk *d_chunks = nullptr, *d_digest_chunks = nullptr;
    uint64_t *d_block_base = nullptr, *d_tensor_ids = nullptr;
    uint32_t *d_seg_count = nullptr;
    unsigned int *d_counter = nullptr;
    unsigned long long *d_status = nullptr;
    uint64_t *d_expected = nullptr;
    bool has_expected = false;
    uint32_t n_segments = 0;
    // chunk list sorted by source offset, for restores fed window by window (built on first use), and the window
    // plans made from it so far, by buffer size
    mutable std::mutex mu;
    mutable Chunk *d_by_src = nullptr;
    mutable std::map<uint64_t, std::vector<gms::SrcWindow>> window_plans;
    const uint64_t *d_src = nullptr, *d_dst = nullptr, *d_len = nullptr;  // the record's columns on the device
};

namespace {

std::atomic<uint64_t> g_launches{0};
thread_local std::string t_cuda_error;

int cuda_fail(cudaError_t e)
{
    t_cuda_error = std::string(cudaGetErrorName(e)) + ": " + cudaGetErrorString(e);
    (void)cudaGetLastError();  // clear the sticky-less error state
    return GMS_ERR_CUDA;
}
#define GMS_CUDA(call)                         \
    do {                                       \
        cudaError_t e_ = (call);               \
        if (e_ != cudaSuccess) return cuda_fail(e_); \
    } while (0)

uint64_t blocks_of(uint64_t nbytes) { return nbytes / gms::kBlockBytes + (nbytes % gms::kBlockBytes ? 1 : 0); }

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// The library's own stream for building tables (one per device, made on first use, never destroyed).  It does not
// synchronise with the default stream, so building a manifest does not wait for whatever else the process has
// queued on the device -- an engine that is still serving, say.
cudaError_t build_stream(cudaStream_t *out)
{
    static std::mutex mu;
    static cudaStream_t streams[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(mu);
    if (!streams[dev] && (e = cudaStreamCreateWithFlags(&streams[dev], cudaStreamNonBlocking)) != cudaSuccess) return e;
    *out = streams[dev];
    return cudaSuccess;
}

// Stable sort of (key, payload) pairs by key.  Validation and list planning sort the tensors' ids, destination and
// source ranges and short-chunk lengths; with tens of thousands of tensors a comparison sort is then most of the
// host's build time, so from a few thousand pairs on this is an LSD radix sort, 11 bits at a time, that skips the
// digits in which all keys agree.
void radix_sort_pairs(std::vector<std::pair<uint64_t, uint64_t>> &v)
{
    if (v.size() < 2048) {
        std::stable_sort(v.begin(), v.end(), [](const auto &a, const auto &b) { return a.first < b.first; });
        return;
    }
    uint64_t all_or = 0, all_and = ~0ull;
    for (const auto &p : v) all_or |= p.first, all_and &= p.first;
    std::vector<std::pair<uint64_t, uint64_t>> tmp(v.size());
    uint32_t count[2049];
    for (int shift = 0; shift < 64; shift += 11) {
        if ((((all_or ^ all_and) >> shift) & 0x7ffu) == 0) continue;  // this digit does not vary
        memset(count, 0, sizeof count);
        for (const auto &p : v) ++count[((p.first >> shift) & 0x7ffu) + 1];
        for (size_t d = 0; d < 2048; ++d) count[d + 1] += count[d];
        for (const auto &p : v) tmp[count[(p.first >> shift) & 0x7ffu]++] = p;
        v.swap(tmp);
    }
}

// Cut every tensor into runs of at most `chunk_blocks` digest blocks.  Large runs first, so that
// the dynamic claim order ends on the small ones and the last wave of warps finishes together.
Chunk make_chunk(const gms_manifest &m, size_t t, uint64_t off, uint64_t n)
{
    const gms_entry &e = m.entries[t];
    Chunk c;
    c.src_off = e.src_offset + off;
    c.dst = reinterpret_cast<uint64_t>(e.dst) + off;
    c.nbytes = (uint32_t)n;
    c.tensor = (uint32_t)t;
    c.gblock0 = (uint32_t)(m.block_base[t] + off / gms::kBlockBytes);
    c.tblock0 = (uint32_t)(off / gms::kBlockBytes);
    return c;
}

// The order is that of a stable sort by length, longest first; since all but the last chunk of a tensor have the full
// length, it is produced directly: the full chunks in entry order, then the tensors' short last chunks sorted among
// themselves (a list of at most one per tensor), instead of sorting a million records.
void build_chunks(const gms_manifest &m, uint32_t chunk_blocks, std::vector<Chunk> &out)
{
    const uint64_t chunk_bytes = (uint64_t)chunk_blocks * gms::kBlockBytes;
    uint64_t n_full = 0, n_tail = 0;
    for (const gms_entry &e : m.entries) {
        n_full += e.nbytes / chunk_bytes;
        n_tail += e.nbytes % chunk_bytes ? 1 : 0;
    }
    out.clear();
    out.resize(n_full + n_tail);
    Chunk *full = out.data(), *tail = out.data() + n_full;
    for (size_t t = 0; t < m.entries.size(); ++t) {
        const gms_entry &e = m.entries[t];
        for (uint64_t off = 0; off < e.nbytes; off += chunk_bytes) {
            const uint64_t n = std::min<uint64_t>(chunk_bytes, e.nbytes - off);
            (n == chunk_bytes ? *full++ : *tail++) = make_chunk(m, t, off, n);
        }
    }
    std::stable_sort(out.begin() + (ptrdiff_t)n_full, out.end(), [](const Chunk &a, const Chunk &b) { return a.nbytes > b.nbytes; });
}

// Where the chunks of each tensor go in a list of the order described above: prefix sums of the full-length chunks,
// and the position of each tensor's short last chunk (ranked by length among the short ones, longest first).
struct ListPlan {
    uint32_t chunk_blocks = 1;
    uint64_t n_full = 0, n_chunks = 0;
    std::vector<uint64_t> full_base;  // n + 1
    std::vector<uint32_t> tail_pos;   // n; 0xffffffff: no short last chunk
};

ListPlan plan_list(const gms_manifest &m, uint32_t chunk_blocks)
{
    const uint64_t chunk_bytes = (uint64_t)chunk_blocks * gms::kBlockBytes;
    const size_t n = m.entries.size();
    ListPlan p;
    p.chunk_blocks = chunk_blocks;
    p.full_base.resize(n + 1);
    p.tail_pos.assign(n, 0xffffffffu);
    // short last chunks ranked by length, longest first, entry order among equals: lengths are below 128 KiB, so the
    // key (chunk_bytes - length) is sorted ascending by the stable radix sort
    std::vector<std::pair<uint64_t, uint64_t>> tails;  // (chunk_bytes - length, tensor)
    uint64_t acc = 0;
    for (size_t t = 0; t < n; ++t) {
        p.full_base[t] = acc;
        acc += m.entries[t].nbytes / chunk_bytes;
        if (m.entries[t].nbytes % chunk_bytes) tails.emplace_back(chunk_bytes - m.entries[t].nbytes % chunk_bytes, t);
    }
    p.full_base[n] = p.n_full = acc;
    radix_sort_pairs(tails);
    for (size_t r = 0; r < tails.size(); ++r) p.tail_pos[tails[r].second] = (uint32_t)(acc + r);
    p.n_chunks = acc + tails.size();
    return p;
}

// Host copies of the two lists, built on first demand (same order as the device writes them in).
void ensure_host_lists(const gms_manifest &m)
{
    std::lock_guard<std::mutex> lock(m.mu);
    if (m.host_lists) return;
    build_chunks(m, m.chunk_blocks, m.chunks);
    build_chunks(m, m.digest_chunk_blocks, m.digest_chunks);
    m.host_lists = true;
}

// Tuning and test hooks read from the environment are honoured only when GMS_TUNING_HOOKS=1 is set as well, so
// that a stray variable in a serving process changes nothing (they are listed in include/gms.h).
long env_hook(const char *name, long lo, long hi, long fallback)
{
    const char *on = getenv("GMS_TUNING_HOOKS");
    if (!on || atoi(on) != 1) return fallback;
    const char *v = getenv(name);
    if (!v) return fallback;
    const long x = atol(v);
    return x >= lo && x <= hi ? x : fallback;
}

int check_kind(const void *image, uint32_t kind)
{
    if (kind != GMS_SRC_DEVICE && kind != GMS_SRC_HOST_MAPPED) return GMS_ERR_KIND;
    cudaPointerAttributes at;
    cudaError_t e = cudaPointerGetAttributes(&at, image);
    if (e != cudaSuccess) return cuda_fail(e);
    if (kind == GMS_SRC_DEVICE && at.type != cudaMemoryTypeDevice && at.type != cudaMemoryTypeManaged) return GMS_ERR_KIND;
    if (kind == GMS_SRC_HOST_MAPPED && at.type != cudaMemoryTypeHost) return GMS_ERR_KIND;
    return GMS_OK;
}

}  // namespace

namespace gms {
uint32_t l2_keep_for(uint64_t n_blocks)
{
    static const long forced = env_hook("GMS_L2_KEEP", 0, 1, -1);  // test hook: 0 = never, 1 = always
    if (forced >= 0) return (uint32_t)forced;
    return n_blocks >= kL2KeepMinBlocks && n_blocks * sizeof(uint64_t) <= kL2KeepBytes ? 1u : 0u;
}
void count_launches(uint32_t n) { g_launches.fetch_add(n, std::memory_order_relaxed); }
int report_cuda_error(cudaError_t e) { return cuda_fail(e); }
}  // namespace gms

namespace gms {

uint64_t manifest_n_tensors(const gms_manifest *m) { return m->entries.size(); }

int manifest_src_windows(const gms_manifest *m, uint64_t buffer_bytes, std::vector<SrcWindow> *out)
{
    if (m->host_only) return GMS_ERR_STATE;
    std::lock_guard<std::mutex> lock(m->mu);
    {
        auto cached = m->window_plans.find(buffer_bytes);  // planned before (the sorted list is on the device by then)
        if (cached != m->window_plans.end()) {
            *out = cached->second;
            return GMS_OK;
        }
    }
    const size_t n = m->entries.size();
    const uint64_t chunk_bytes = (uint64_t)m->chunk_blocks * kBlockBytes;
    // the copy list in order of source offset: the tensors in order of their offsets, each one's chunks in order
    std::vector<uint32_t> order(n);
    std::iota(order.begin(), order.end(), 0u);
    std::stable_sort(order.begin(), order.end(),
                     [&](uint32_t a, uint32_t b) { return m->entries[a].src_offset < m->entries[b].src_offset; });
    std::vector<Chunk> sorted;  // only when tensors share image bytes: then the chunks themselves have to be sorted
    if (!m->sources_disjoint) {
        sorted.reserve(m->n_chunks);
        for (uint32_t t : order)
            for (uint64_t off = 0; off < m->entries[t].nbytes; off += chunk_bytes)
                sorted.push_back(make_chunk(*m, t, off, std::min<uint64_t>(chunk_bytes, m->entries[t].nbytes - off)));
        std::stable_sort(sorted.begin(), sorted.end(), [](const Chunk &a, const Chunk &b) { return a.src_off < b.src_off; });
    }
    if (!m->d_by_src && m->n_chunks) {
        cudaError_t e = cudaMalloc(&m->d_by_src, (size_t)m->n_chunks * sizeof(Chunk));
        if (e != cudaSuccess) {
            (void)cudaGetLastError();
            return e == cudaErrorMemoryAllocation ? GMS_ERR_NOMEM : cuda_fail(e);
        }
        if (m->sources_disjoint) {
            // written on the device like the other lists: every tensor's chunks, its short last one included, in place
            std::vector<uint64_t> base(n + 1);
            uint64_t acc = 0;
            for (size_t k = 0; k < n; ++k) {
                base[k] = acc;
                acc += (m->entries[order[k]].nbytes + chunk_bytes - 1) / chunk_bytes;
            }
            base[n] = acc;
            const size_t o_perm = (n + 1) * sizeof(uint64_t), o_tail = o_perm + n * sizeof(uint32_t), bytes = o_tail + n * sizeof(uint32_t);
            std::vector<uint8_t> h(bytes, 0xff);  // tail positions: all "none"
            memcpy(h.data(), base.data(), (n + 1) * sizeof(uint64_t));
            if (n) memcpy(h.data() + o_perm, order.data(), n * sizeof(uint32_t));
            uint8_t *tmp = nullptr;
            cudaStream_t bs = nullptr;
            e = build_stream(&bs);
            if (e == cudaSuccess) e = cudaMalloc(&tmp, bytes);
            if (e == cudaSuccess) e = cudaMemcpyAsync(tmp, h.data(), bytes, cudaMemcpyHostToDevice, bs);
            ExpandArgs x;
            x.src_offset = m->d_src;
            x.dst = m->d_dst;
            x.nbytes = m->d_len;
            x.block_base = m->d_block_base;
            x.full_base = reinterpret_cast<const uint64_t *>(tmp);
            x.perm = reinterpret_cast<const uint32_t *>(tmp + o_perm);
            x.tail_pos = reinterpret_cast<const uint32_t *>(tmp + o_tail);
            x.n_tensors = (uint32_t)n;
            x.n_full = acc;
            x.chunk_blocks = m->chunk_blocks;
            x.out = m->d_by_src;
            if (e == cudaSuccess) e = launch_expand_chunks(x, bs);
            if (e == cudaSuccess) e = cudaStreamSynchronize(bs);
            if (tmp) cudaFree(tmp);
        } else {
            e = cudaMemcpy(m->d_by_src, sorted.data(), sorted.size() * sizeof(Chunk), cudaMemcpyHostToDevice);
        }
        if (e != cudaSuccess) {
            cudaFree(m->d_by_src);
            m->d_by_src = nullptr;
            return cuda_fail(e);
        }
    }
    // greedy cut: a window takes chunks, in list order, while their sources span at most one buffer
    out->clear();
    size_t ti = 0;          // cursor: tensor slot in `order` ...
    uint64_t off = 0;       // ... and byte offset of the next chunk inside it (disjoint sources), or
    size_t si = 0;          // index into `sorted` (shared sources)
    auto skip_empty = [&] {
        while (ti < n && off >= m->entries[order[ti]].nbytes) ++ti, off = 0;
    };
    skip_empty();
    uint64_t i = 0;
    while (i < m->n_chunks) {
        SrcWindow w;
        w.first_chunk = (uint32_t)i;
        const uint64_t first = i;
        bool started = false;
        w.src_lo = w.src_hi = 0;
        while (i < m->n_chunks) {
            uint64_t src, len;
            if (m->sources_disjoint) {
                const gms_entry &e = m->entries[order[ti]];
                src = e.src_offset + off;
                len = std::min<uint64_t>(chunk_bytes, e.nbytes - off);
            } else {
                src = sorted[si].src_off;
                len = sorted[si].nbytes;
            }
            if (!started) w.src_lo = w.src_hi = src, started = true;
            const uint64_t end = src + len;
            if (std::max(end, w.src_hi) - w.src_lo > buffer_bytes) break;
            w.src_hi = std::max(end, w.src_hi);
            ++i;
            if (m->sources_disjoint) {
                off += chunk_bytes;
                skip_empty();
            } else {
                ++si;
            }
        }
        if (i == first) return GMS_ERR_ARG;  // a single chunk does not fit the buffer
        w.n_chunks = (uint32_t)(i - first);
        out->push_back(w);
    }
    m->window_plans[buffer_bytes] = *out;
    return GMS_OK;
}

int manifest_sorted_sources(const gms_manifest *m, std::vector<std::pair<uint64_t, uint64_t>> *out)
{
    if (!m->sources_disjoint) return GMS_ERR_OVERLAP;
    out->clear();
    for (const gms_entry &e : m->entries)
        if (e.nbytes) out->emplace_back(e.src_offset, e.nbytes);
    std::sort(out->begin(), out->end());
    return GMS_OK;
}

int manifest_launch_window(const gms_manifest *m, const SrcWindow &w, const void *window_base, bool first,
                           uint64_t *d_block_digests, uint64_t *d_tensor_digests, cudaStream_t s, bool capture)
{
    StreamArgs a;
    a.chunks = m->d_by_src + w.first_chunk;
    a.n_chunks = w.n_chunks;
    a.image = static_cast<const uint8_t *>(window_base) - w.src_lo;  // so that image + src_off lands in the window
    a.block_digests = d_block_digests;
    a.tensor_digests = d_tensor_digests;
    a.n_tensors = (uint32_t)m->entries.size();
    a.work_counters = m->d_counter;
    a.status = m->d_status;
    a.n_counters = 1;
    a.group = 1;
    a.capture = capture ? 1u : 0u;
    a.keep_accum = first ? 0u : 1u;
    a.stall_chunk = 0xffffffffu;
    a.expected = nullptr;
    a.seg_count = nullptr;
    a.n_segments = 0;
    a.l2_keep = 0;
    cudaError_t e = launch_restore(a, s);
    return e == cudaSuccess ? GMS_OK : cuda_fail(e);
}

}  // namespace gms

extern "C" {

int gms_manifest_build(const gms_entry *entries, size_t n, uint64_t image_bytes, uint32_t flags, gms_manifest **out)
{
    if (!out || (n && !entries)) return GMS_ERR_NULL;
    *out = nullptr;
    if (flags & ~(GMS_BUILD_HOST_ONLY | GMS_BUILD_SELFTEST_STALL)) return GMS_ERR_ARG;
    if (n >= 0xffffffffull) return GMS_ERR_RANGE;

    // ---- validation (all on the host, before any CUDA call)
    uint64_t n_blocks = 0, payload = 0;
    for (size_t t = 0; t < n; ++t) {
        const gms_entry &e = entries[t];
        if ((e.src_offset & 15u) || (reinterpret_cast<uint64_t>(e.dst) & 15u)) return GMS_ERR_ALIGN;
        if (e.nbytes && !e.dst) return GMS_ERR_NULL;
        if (e.src_offset > image_bytes || e.nbytes > image_bytes - e.src_offset) return GMS_ERR_RANGE;
        if (reinterpret_cast<uint64_t>(e.dst) + e.nbytes < reinterpret_cast<uint64_t>(e.dst)) return GMS_ERR_RANGE;
        n_blocks += blocks_of(e.nbytes);
        payload += e.nbytes;
        if (n_blocks >= 0xffffffffull) return GMS_ERR_RANGE;  // digest slots are indexed with 32 bits on the device
    }
    gms_manifest *m = nullptr;
    try {
        // the three checks sort plain key arrays (ids; (start, end) of destinations; (start, end) of sources): with ten
        // thousand tensors that is a few hundred microseconds each, where sorting indices into the records took over a
        // millisecond each
        std::vector<std::pair<uint64_t, uint64_t>> span(n);
        for (size_t t = 0; t < n; ++t) span[t] = {entries[t].tensor_id, 0};
        radix_sort_pairs(span);
        for (size_t i = 1; i < n; ++i)
            if (span[i].first == span[i - 1].first) return GMS_ERR_DUP_ID;
        // destinations pairwise disjoint: sort the non-empty ones by address, compare neighbours (with equal starts
        // any order will do: two non-empty ranges that start together overlap)
        span.clear();
        for (size_t t = 0; t < n; ++t)
            if (entries[t].nbytes) span.emplace_back(reinterpret_cast<uint64_t>(entries[t].dst), reinterpret_cast<uint64_t>(entries[t].dst) + entries[t].nbytes);
        radix_sort_pairs(span);
        for (size_t i = 1; i < span.size(); ++i)
            if (span[i - 1].second > span[i].first) return GMS_ERR_OVERLAP;

        bool sources_disjoint = true;
        span.clear();
        for (size_t t = 0; t < n; ++t)
            if (entries[t].nbytes) span.emplace_back(entries[t].src_offset, entries[t].src_offset + entries[t].nbytes);
        radix_sort_pairs(span);
        for (size_t i = 1; i < span.size(); ++i)
            if (span[i - 1].second > span[i].first) sources_disjoint = false;

        m = new gms_manifest();
        m->sources_disjoint = sources_disjoint;
        m->entries.assign(entries, entries + n);
        m->image_bytes = image_bytes;
        m->payload = payload;
        m->n_blocks = n_blocks;
        m->host_only = (flags & GMS_BUILD_HOST_ONLY) != 0;
        m->selftest_stall = (flags & GMS_BUILD_SELFTEST_STALL) != 0;
        m->block_base.resize(n + 1);
        uint64_t acc = 0;
        for (size_t t = 0; t < n; ++t) {
            m->block_base[t] = acc;
            acc += blocks_of(entries[t].nbytes);
        }
        m->block_base[n] = acc;

        // ---- chunk length (needs the number of warps the restore kernel runs; a B200's if no device is asked)
        uint32_t total_warps = 148 * 9, digest_warps = 148 * 16;
        if (!m->host_only) {
            gms::Geometry g;
            cudaError_t e = gms::get_geometry(gms::kRestore, &g);
            if (e != cudaSuccess) {
                delete m;
                return cuda_fail(e);
            }
            total_warps = g.grid * g.warps;
            if ((e = gms::get_geometry(gms::kDigest, &g)) != cudaSuccess) {
                delete m;
                return cuda_fail(e);
            }
            digest_warps = g.grid * g.warps;
            (void)cudaGetDevice(&m->device);
        }
        // Chunk length: 4 blocks (16 KiB).  Claims are made in strict list order, so short chunks keep all bytes in
        // flight within a narrow moving window of the image, which HBM rewards; shorter than 4 and the per-chunk
        // work shows.  Manifests too small to give every warp two such chunks are cut finer.
        uint32_t chunk_blocks = (uint32_t)std::min<uint64_t>(4, std::max<uint64_t>(1, (n_blocks + 2ull * total_warps - 1) / (2ull * total_warps)));
        chunk_blocks = (uint32_t)env_hook("GMS_CHUNK_BLOCKS", 1, gms::kMaxChunkBlocks, chunk_blocks);
        m->chunk_blocks = chunk_blocks;
        // The digest-only kernel reads twice as fast as the restore kernel moves payload and has no store side to
        // keep narrow: it is fastest on runs of 8 blocks (32 KiB) -- 2.25 ms against 2.40 ms with 4-block chunks on
        // a 16 GB manifest -- while the restore slows down on anything longer than 4.  So it gets a list of its own.
        uint32_t digest_blocks = (uint32_t)std::min<uint64_t>(8, std::max<uint64_t>(1, (n_blocks + 2ull * digest_warps - 1) / (2ull * digest_warps)));
        digest_blocks = (uint32_t)env_hook("GMS_CHUNK_BLOCKS_DIGEST", 1, gms::kMaxChunkBlocks, digest_blocks);
        m->digest_chunk_blocks = digest_blocks;
        const ListPlan plan = plan_list(*m, chunk_blocks), dplan = plan_list(*m, digest_blocks);
        m->n_chunks = plan.n_chunks;
        m->n_digest_chunks = dplan.n_chunks;
        m->n_segments = (uint32_t)((n_blocks + gms::kVerifySegBlocks - 1) / gms::kVerifySegBlocks);

        // ---- device tables: the per-tensor columns go up in one copy, the chunk lists are written by a kernel each
        if (!m->host_only) {
            const size_t o_chunks = 0;
            const size_t o_dchunks = align_up(o_chunks + (size_t)m->n_chunks * sizeof(Chunk), 256);
            const size_t o_base = align_up(o_dchunks + (size_t)m->n_digest_chunks * sizeof(Chunk), 256);
            const size_t o_ids = align_up(o_base + (n + 1) * sizeof(uint64_t), 256);
            const size_t o_src = align_up(o_ids + n * sizeof(uint64_t), 256);
            const size_t o_dst = align_up(o_src + n * sizeof(uint64_t), 256);
            const size_t o_len = align_up(o_dst + n * sizeof(uint64_t), 256);
            const size_t o_fb = align_up(o_len + n * sizeof(uint64_t), 256);
            const size_t o_dfb = align_up(o_fb + (n + 1) * sizeof(uint64_t), 256);
            const size_t o_tp = align_up(o_dfb + (n + 1) * sizeof(uint64_t), 256);
            const size_t o_dtp = align_up(o_tp + n * sizeof(uint32_t), 256);
            const size_t o_segcnt = align_up(o_dtp + n * sizeof(uint32_t), 256);
            const size_t o_ctr = align_up(o_segcnt + (size_t)m->n_segments * sizeof(uint32_t), 256);
            const size_t o_status = o_ctr + (size_t)gms::kMaxCounters * gms::kCounterStride * sizeof(unsigned int);
            const size_t total = o_status + 128;
            std::vector<uint8_t> h(o_segcnt - o_base, 0);  // the columns: a few dozen bytes per tensor
            uint8_t *hp = h.data() - o_base;                // so that hp + o_x addresses column x
            memcpy(hp + o_base, m->block_base.data(), (n + 1) * sizeof(uint64_t));
            for (size_t t = 0; t < n; ++t) {
                const uint64_t dst = reinterpret_cast<uint64_t>(entries[t].dst);
                memcpy(hp + o_ids + t * 8, &entries[t].tensor_id, 8);
                memcpy(hp + o_src + t * 8, &entries[t].src_offset, 8);
                memcpy(hp + o_dst + t * 8, &dst, 8);
                memcpy(hp + o_len + t * 8, &entries[t].nbytes, 8);
            }
            memcpy(hp + o_fb, plan.full_base.data(), (n + 1) * sizeof(uint64_t));
            memcpy(hp + o_dfb, dplan.full_base.data(), (n + 1) * sizeof(uint64_t));
            if (n) memcpy(hp + o_tp, plan.tail_pos.data(), n * sizeof(uint32_t));
            if (n) memcpy(hp + o_dtp, dplan.tail_pos.data(), n * sizeof(uint32_t));
            cudaError_t e = cudaMalloc(&m->d_tables, total);
            if (e != cudaSuccess) {
                delete m;
                (void)cudaGetLastError();
                return e == cudaErrorMemoryAllocation ? GMS_ERR_NOMEM : cuda_fail(e);
            }
            m->d_chunks = reinterpret_cast<Chunk *>(m->d_tables + o_chunks);
            m->d_digest_chunks = reinterpret_cast<Chunk *>(m->d_tables + o_dchunks);
            m->d_block_base = reinterpret_cast<uint64_t *>(m->d_tables + o_base);
            m->d_tensor_ids = reinterpret_cast<uint64_t *>(m->d_tables + o_ids);
            m->d_seg_count = reinterpret_cast<uint32_t *>(m->d_tables + o_segcnt);
            m->d_counter = reinterpret_cast<unsigned int *>(m->d_tables + o_ctr);
            m->d_status = reinterpret_cast<unsigned long long *>(m->d_tables + o_status);
            cudaStream_t bs = nullptr;
            e = build_stream(&bs);
            if (e == cudaSuccess) e = cudaMemcpyAsync(m->d_tables + o_base, h.data(), h.size(), cudaMemcpyHostToDevice, bs);
            if (e == cudaSuccess) e = cudaMemsetAsync(m->d_tables + o_segcnt, 0, total - o_segcnt, bs);
            gms::ExpandArgs x;
            x.src_offset = m->d_src = reinterpret_cast<const uint64_t *>(m->d_tables + o_src);
            x.dst = m->d_dst = reinterpret_cast<const uint64_t *>(m->d_tables + o_dst);
            x.nbytes = m->d_len = reinterpret_cast<const uint64_t *>(m->d_tables + o_len);
            x.perm = nullptr;
            x.block_base = m->d_block_base;
            x.n_tensors = (uint32_t)n;
            x.full_base = reinterpret_cast<const uint64_t *>(m->d_tables + o_fb);
            x.tail_pos = reinterpret_cast<const uint32_t *>(m->d_tables + o_tp);
            x.n_full = plan.n_full;
            x.chunk_blocks = chunk_blocks;
            x.out = m->d_chunks;
            if (e == cudaSuccess) e = gms::launch_expand_chunks(x, bs);
            x.full_base = reinterpret_cast<const uint64_t *>(m->d_tables + o_dfb);
            x.tail_pos = reinterpret_cast<const uint32_t *>(m->d_tables + o_dtp);
            x.n_full = dplan.n_full;
            x.chunk_blocks = digest_blocks;
            x.out = m->d_digest_chunks;
            if (e == cudaSuccess) e = gms::launch_expand_chunks(x, bs);
            if (e == cudaSuccess) e = cudaStreamSynchronize(bs);  // the lists are complete when the call returns
            if (e == cudaSuccess && env_hook("GMS_CHECK_TABLES", 0, 1, 0)) {
                // test hook: the device-written lists must equal the host's construction of the same order
                ensure_host_lists(*m);
                std::vector<Chunk> got(m->n_chunks + m->n_digest_chunks);
                e = cudaMemcpy(got.data(), m->d_chunks, (size_t)m->n_chunks * sizeof(Chunk), cudaMemcpyDeviceToHost);
                if (e == cudaSuccess)
                    e = cudaMemcpy(got.data() + m->n_chunks, m->d_digest_chunks, (size_t)m->n_digest_chunks * sizeof(Chunk),
                                   cudaMemcpyDeviceToHost);
                const bool same = e == cudaSuccess && m->chunks.size() == m->n_chunks && m->digest_chunks.size() == m->n_digest_chunks &&
                                  (m->n_chunks == 0 || memcmp(got.data(), m->chunks.data(), (size_t)m->n_chunks * sizeof(Chunk)) == 0) &&
                                  (m->n_digest_chunks == 0 || memcmp(got.data() + m->n_chunks, m->digest_chunks.data(),
                                                                     (size_t)m->n_digest_chunks * sizeof(Chunk)) == 0);
                if (e == cudaSuccess && !same) {
                    cudaFree(m->d_tables);
                    delete m;
                    return GMS_ERR_STATE;
                }
            }
            if (e != cudaSuccess) {
                cudaFree(m->d_tables);
                delete m;
                return cuda_fail(e);
            }
        }
        *out = m;
        return GMS_OK;
    } catch (const std::bad_alloc &) {
        if (m) {
            if (m->d_tables) cudaFree(m->d_tables);
            delete m;
        }
        return GMS_ERR_NOMEM;
    }
}

int gms_manifest_destroy(gms_manifest *m)
{
    if (!m) return GMS_OK;
    int rc = GMS_OK;
    if (m->d_expected && cudaFree(m->d_expected) != cudaSuccess) rc = GMS_ERR_CUDA;
    if (m->d_tables && cudaFree(m->d_tables) != cudaSuccess) rc = GMS_ERR_CUDA;
    if (m->d_by_src && cudaFree(m->d_by_src) != cudaSuccess) rc = GMS_ERR_CUDA;
    delete m;
    return rc;
}

int gms_manifest_info(const gms_manifest *m, uint64_t *n_tensors, uint64_t *n_blocks, uint64_t *payload_bytes)
{
    if (!m) return GMS_ERR_NULL;
    if (n_tensors) *n_tensors = m->entries.size();
    if (n_blocks) *n_blocks = m->n_blocks;
    if (payload_bytes) *payload_bytes = m->payload;
    return GMS_OK;
}

int gms_manifest_block_base(const gms_manifest *m, size_t entry_index, uint64_t *first_block)
{
    if (!m || !first_block) return GMS_ERR_NULL;
    if (entry_index >= m->entries.size()) return GMS_ERR_ARG;
    *first_block = m->block_base[entry_index];
    return GMS_OK;
}

int gms_manifest_chunk_count(const gms_manifest *m, uint64_t *n_chunks)
{
    if (!m || !n_chunks) return GMS_ERR_NULL;
    *n_chunks = m->n_chunks;
    return GMS_OK;
}

int gms_manifest_chunk(const gms_manifest *m, uint64_t i, uint64_t *entry_index, uint64_t *tensor_byte_offset, uint64_t *nbytes)
{
    if (!m) return GMS_ERR_NULL;
    if (i >= m->n_chunks) return GMS_ERR_ARG;
    try {
        ensure_host_lists(*m);
    } catch (const std::bad_alloc &) {
        return GMS_ERR_NOMEM;
    }
    const Chunk &c = m->chunks[i];
    if (entry_index) *entry_index = c.tensor;
    if (tensor_byte_offset) *tensor_byte_offset = (uint64_t)c.tblock0 * gms::kBlockBytes;
    if (nbytes) *nbytes = c.nbytes;
    return GMS_OK;
}

int gms_manifest_set_expected(gms_manifest *m, const uint64_t *d_block_digests, void *stream)
{
    if (!m || (m->n_blocks && !d_block_digests)) return GMS_ERR_NULL;
    if (m->host_only) return GMS_ERR_STATE;
    if (!m->d_expected && m->n_blocks) {
        cudaError_t e = cudaMalloc(&m->d_expected, m->n_blocks * sizeof(uint64_t));
        if (e != cudaSuccess) {
            (void)cudaGetLastError();
            return e == cudaErrorMemoryAllocation ? GMS_ERR_NOMEM : cuda_fail(e);
        }
    }
    GMS_CUDA(gms::launch_copy_u64(m->d_expected, d_block_digests, m->n_blocks, static_cast<cudaStream_t>(stream)));
    m->has_expected = true;
    return GMS_OK;
}

static int stream_call(const gms_manifest *m, const void *image, bool store, uint64_t *d_block_digests,
                       uint64_t *d_tensor_digests, void *stream, bool capture = false, bool compare = false)
{
    gms::StreamArgs a;
    a.chunks = store ? m->d_chunks : m->d_digest_chunks;
    a.n_chunks = (uint32_t)(store ? m->n_chunks : m->n_digest_chunks);
    a.image = static_cast<const uint8_t *>(image);
    a.block_digests = d_block_digests;
    a.tensor_digests = d_tensor_digests;
    a.n_tensors = (uint32_t)m->entries.size();
    a.work_counters = m->d_counter;
    a.status = m->d_status;
    a.n_counters = 1;
    a.group = 1;
    a.capture = capture ? 1u : 0u;
    a.keep_accum = 0;
    a.stall_chunk = m->selftest_stall ? 0u : 0xffffffffu;
    a.expected = compare ? m->d_expected : nullptr;
    a.seg_count = compare ? m->d_seg_count : nullptr;
    a.n_segments = compare ? m->n_segments : 0;
    a.l2_keep = store ? 0u : gms::l2_keep_for(m->n_blocks);
    GMS_CUDA(store ? gms::launch_restore(a, static_cast<cudaStream_t>(stream))
                   : gms::launch_digest(a, static_cast<cudaStream_t>(stream)));
    return GMS_OK;
}

int gms_restore(const gms_manifest *m, const void *image, uint32_t image_kind, uint64_t *d_block_digests,
                uint64_t *d_tensor_digests, void *stream)
{
    if (!m || (!image && m->payload)) return GMS_ERR_NULL;
    if (image_kind != GMS_SRC_DEVICE && image_kind != GMS_SRC_HOST_MAPPED) return GMS_ERR_KIND;
    if (reinterpret_cast<uint64_t>(image) & 15u) return GMS_ERR_ALIGN;
    if (m->host_only) return GMS_ERR_STATE;
    if (image) {
        const int rc = check_kind(image, image_kind);
        if (rc) return rc;
    }
    return stream_call(m, image, true, d_block_digests, d_tensor_digests, stream);
}

int gms_capture(const gms_manifest *m, void *image, uint32_t image_kind, uint64_t *d_block_digests,
                uint64_t *d_tensor_digests, void *stream)
{
    if (!m || (!image && m->payload)) return GMS_ERR_NULL;
    if (image_kind != GMS_SRC_DEVICE && image_kind != GMS_SRC_HOST_MAPPED) return GMS_ERR_KIND;
    if (reinterpret_cast<uint64_t>(image) & 15u) return GMS_ERR_ALIGN;
    if (!m->sources_disjoint) return GMS_ERR_OVERLAP;
    if (m->host_only) return GMS_ERR_STATE;
    if (image) {
        const int rc = check_kind(image, image_kind);
        if (rc) return rc;
    }
    return stream_call(m, image, true, d_block_digests, d_tensor_digests, stream, true);
}

int gms_digest(const gms_manifest *m, uint64_t *d_block_digests, uint64_t *d_tensor_digests, void *stream)
{
    if (!m) return GMS_ERR_NULL;
    if (m->host_only) return GMS_ERR_STATE;
    return stream_call(m, nullptr, false, d_block_digests, d_tensor_digests, stream);
}

int gms_verify(const gms_manifest *m, const uint64_t *d_block_digests, gms_mismatch *d_out, uint32_t cap, uint64_t *d_count,
               void *stream)
{
    if (!m || !d_count || (cap && !d_out) || (m->n_blocks && !d_block_digests)) return GMS_ERR_NULL;
    if (m->host_only || !m->has_expected) return GMS_ERR_STATE;
    gms::VerifyArgs a = {};
    a.computed = d_block_digests;
    a.expected = m->d_expected;
    a.n_blocks = m->n_blocks;
    a.block_base = m->d_block_base;
    a.tensor_ids = m->d_tensor_ids;
    a.n_tensors = (uint32_t)m->entries.size();
    a.seg_count = m->d_seg_count;
    a.n_segments = m->n_segments;
    a.out = d_out;
    a.cap = cap;
    a.count = d_count;
    GMS_CUDA(gms::launch_verify(a, static_cast<cudaStream_t>(stream)));
    return GMS_OK;
}

// The streaming kernel has counted the differing slots of every segment; only the ordered emit is left.
static int verify_counted(const gms_manifest *m, const uint64_t *d_block_digests, gms_mismatch *d_out, uint32_t cap,
                          uint64_t *d_count, void *stream)
{
    gms::VerifyArgs a = {};
    a.computed = d_block_digests;
    a.expected = m->d_expected;
    a.n_blocks = m->n_blocks;
    a.block_base = m->d_block_base;
    a.tensor_ids = m->d_tensor_ids;
    a.n_tensors = (uint32_t)m->entries.size();
    a.seg_count = m->d_seg_count;
    a.n_segments = m->n_segments;
    a.out = d_out;
    a.cap = cap;
    a.count = d_count;
    GMS_CUDA(gms::launch_verify_counted(a, static_cast<cudaStream_t>(stream)));
    return GMS_OK;
}

int gms_digest_verify(const gms_manifest *m, uint64_t *d_block_digests, uint64_t *d_tensor_digests, gms_mismatch *d_out,
                      uint32_t cap, uint64_t *d_count, void *stream)
{
    if (!m || !d_count || (cap && !d_out) || (m->n_blocks && !d_block_digests)) return GMS_ERR_NULL;
    if (m->host_only || !m->has_expected) return GMS_ERR_STATE;
    const int rc = stream_call(m, nullptr, false, d_block_digests, d_tensor_digests, stream, false, true);
    return rc ? rc : verify_counted(m, d_block_digests, d_out, cap, d_count, stream);
}

int gms_restore_verify(const gms_manifest *m, const void *image, uint32_t image_kind, uint64_t *d_block_digests,
                       uint64_t *d_tensor_digests, gms_mismatch *d_out, uint32_t cap, uint64_t *d_count, void *stream)
{
    if (!m || (!image && m->payload) || !d_count || (cap && !d_out) || (m->n_blocks && !d_block_digests)) return GMS_ERR_NULL;
    if (image_kind != GMS_SRC_DEVICE && image_kind != GMS_SRC_HOST_MAPPED) return GMS_ERR_KIND;
    if (reinterpret_cast<uint64_t>(image) & 15u) return GMS_ERR_ALIGN;
    if (m->host_only || !m->has_expected) return GMS_ERR_STATE;
    if (image) {
        const int rc = check_kind(image, image_kind);
        if (rc) return rc;
    }
    const int rc = stream_call(m, image, true, d_block_digests, d_tensor_digests, stream, false, true);
    return rc ? rc : verify_counted(m, d_block_digests, d_out, cap, d_count, stream);
}

int gms_verify_tensors(const gms_manifest *m, const uint64_t *d_block_digests, uint32_t *d_tensor_counts, void *stream)
{
    if (!m || (m->n_blocks && !d_block_digests) || (!m->entries.empty() && !d_tensor_counts)) return GMS_ERR_NULL;
    if (m->host_only || !m->has_expected) return GMS_ERR_STATE;
    gms::VerifyArgs a = {};
    a.computed = d_block_digests;
    a.expected = m->d_expected;
    a.n_blocks = m->n_blocks;
    a.block_base = m->d_block_base;
    a.tensor_ids = m->d_tensor_ids;
    a.n_tensors = (uint32_t)m->entries.size();
    GMS_CUDA(gms::launch_verify_tensor_counts(a, d_tensor_counts, static_cast<cudaStream_t>(stream)));
    return GMS_OK;
}

int gms_last_device_status(const gms_manifest *m, void *stream, uint64_t *word)
{
    if (!m || !word) return GMS_ERR_NULL;
    if (m->host_only) return GMS_ERR_STATE;
    unsigned long long w = 0;
    GMS_CUDA(cudaMemcpyAsync(&w, m->d_status, sizeof w, cudaMemcpyDeviceToHost, static_cast<cudaStream_t>(stream)));
    GMS_CUDA(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
    *word = w;
    return (w & GMS_DEV_TIMEOUT) ? GMS_ERR_TIMEOUT : GMS_OK;
}

// A plane spans (n_blocks - 1) * block_stride + block_bytes bytes; with more than one plane, a smaller plane stride
// would make planes share bytes, and a scatter into shared bytes has no defined result.
static bool planes_overlap(const gms_kv_pool *pool)
{
    if (pool->n_planes < 2 || pool->n_blocks == 0) return false;
    return pool->plane_stride < (uint64_t)(pool->n_blocks - 1) * pool->block_stride + pool->block_bytes;
}

static int kv_call(const gms_kv_pool *pool, const void *image, uint64_t img_plane_stride, uint64_t img_slot_stride,
                   uint32_t image_kind, const int32_t *d_block_ids, uint32_t n_sel, uint64_t *d_block_digests,
                   uint64_t *d_kv_digests, uint64_t *d_status, void *stream, bool capture)
{
    if (!pool || !d_status) return GMS_ERR_NULL;
    if (image_kind != GMS_SRC_DEVICE && image_kind != GMS_SRC_HOST_MAPPED) return GMS_ERR_KIND;
    if (pool->block_bytes == 0 || pool->block_bytes % gms::kBlockBytes) return GMS_ERR_ALIGN;
    if (pool->block_bytes > gms::kMaxChunkBlocks * gms::kBlockBytes) return GMS_ERR_ARG;
    const bool work = n_sel && pool->n_planes;
    if (work && (!pool->base || !image || !d_block_ids)) return GMS_ERR_NULL;
    if ((reinterpret_cast<uint64_t>(pool->base) | reinterpret_cast<uint64_t>(image) | pool->plane_stride | pool->block_stride |
         img_plane_stride | img_slot_stride) & 15u)
        return GMS_ERR_ALIGN;
    if (pool->block_stride < pool->block_bytes && pool->n_blocks > 1) return GMS_ERR_ARG;
    if (planes_overlap(pool)) return GMS_ERR_ARG;
    if (pool->flags & ~GMS_KV_IMAGE_BY_ID) return GMS_ERR_ARG;
    const uint64_t k = pool->block_bytes / gms::kBlockBytes;
    if ((uint64_t)n_sel * pool->n_planes * k >= 0xffffffffull) return GMS_ERR_RANGE;
    if (work) {
        const int rc = check_kind(image, image_kind);
        if (rc) return rc;
    }
    gms::KvArgs a;
    a.pool_base = static_cast<uint8_t *>(pool->base);
    a.plane_stride = pool->plane_stride;
    a.block_stride = pool->block_stride;
    a.n_planes = pool->n_planes;
    a.n_blocks = pool->n_blocks;
    a.block_bytes = pool->block_bytes;
    a.image = static_cast<const uint8_t *>(image);
    a.img_plane_stride = img_plane_stride;
    a.img_slot_stride = img_slot_stride;
    a.ids = d_block_ids;
    a.n_sel = n_sel;
    a.block_digests = d_block_digests;
    a.kv_digests = d_kv_digests;
    a.status = reinterpret_cast<unsigned long long *>(d_status);
    a.capture = capture ? 1u : 0u;
    a.digest_only = 0u;
    a.by_id = (pool->flags & GMS_KV_IMAGE_BY_ID) ? 1u : 0u;
    a.l2_keep = 0u;
    GMS_CUDA(gms::launch_kv_restore(a, static_cast<cudaStream_t>(stream)));
    return GMS_OK;
}

int gms_kv_restore(const gms_kv_pool *pool, const void *image, uint64_t img_plane_stride, uint64_t img_slot_stride,
                   uint32_t image_kind, const int32_t *d_block_ids, uint32_t n_sel, uint64_t *d_block_digests,
                   uint64_t *d_kv_digests, uint64_t *d_status, void *stream)
{
    return kv_call(pool, image, img_plane_stride, img_slot_stride, image_kind, d_block_ids, n_sel, d_block_digests, d_kv_digests,
                   d_status, stream, false);
}

int gms_kv_capture(const gms_kv_pool *pool, void *image, uint64_t img_plane_stride, uint64_t img_slot_stride,
                   uint32_t image_kind, const int32_t *d_block_ids, uint32_t n_sel, uint64_t *d_block_digests,
                   uint64_t *d_kv_digests, uint64_t *d_status, void *stream)
{
    return kv_call(pool, image, img_plane_stride, img_slot_stride, image_kind, d_block_ids, n_sel, d_block_digests, d_kv_digests,
                   d_status, stream, true);
}

int gms_kv_digest(const gms_kv_pool *pool, const int32_t *d_block_ids, uint32_t n_sel, uint64_t *d_block_digests,
                  uint64_t *d_kv_digests, uint64_t *d_status, void *stream)
{
    if (!pool || !d_status) return GMS_ERR_NULL;
    if (pool->block_bytes == 0 || pool->block_bytes % gms::kBlockBytes) return GMS_ERR_ALIGN;
    if (pool->block_bytes > gms::kMaxChunkBlocks * gms::kBlockBytes) return GMS_ERR_ARG;
    const bool work = n_sel && pool->n_planes;
    if (work && (!pool->base || !d_block_ids)) return GMS_ERR_NULL;
    if ((reinterpret_cast<uint64_t>(pool->base) | pool->plane_stride | pool->block_stride) & 15u) return GMS_ERR_ALIGN;
    if (pool->block_stride < pool->block_bytes && pool->n_blocks > 1) return GMS_ERR_ARG;
    if (planes_overlap(pool)) return GMS_ERR_ARG;
    if (pool->flags & ~GMS_KV_IMAGE_BY_ID) return GMS_ERR_ARG;
    const uint64_t k = pool->block_bytes / gms::kBlockBytes;
    if ((uint64_t)n_sel * pool->n_planes * k >= 0xffffffffull) return GMS_ERR_RANGE;
    gms::KvArgs a = {};
    a.pool_base = static_cast<uint8_t *>(pool->base);
    a.plane_stride = pool->plane_stride;
    a.block_stride = pool->block_stride;
    a.n_planes = pool->n_planes;
    a.n_blocks = pool->n_blocks;
    a.block_bytes = pool->block_bytes;
    a.ids = d_block_ids;
    a.n_sel = n_sel;
    a.block_digests = d_block_digests;
    a.kv_digests = d_kv_digests;
    a.status = reinterpret_cast<unsigned long long *>(d_status);
    a.digest_only = 1u;
    a.l2_keep = gms::l2_keep_for((uint64_t)n_sel * pool->n_planes * k);
    GMS_CUDA(gms::launch_kv_restore(a, static_cast<cudaStream_t>(stream)));
    return GMS_OK;
}

int gms_kv_verify(const gms_kv_pool *pool, const int32_t *d_block_ids, uint32_t n_sel, const uint64_t *d_computed,
                  const uint64_t *d_expected, gms_kv_mismatch *d_out, uint32_t cap, uint64_t *d_count, uint32_t *d_scratch,
                  void *stream)
{
    if (!pool || !d_count || (cap && !d_out)) return GMS_ERR_NULL;
    if (pool->block_bytes == 0 || pool->block_bytes % gms::kBlockBytes) return GMS_ERR_ALIGN;
    if (pool->block_bytes > gms::kMaxChunkBlocks * gms::kBlockBytes) return GMS_ERR_ARG;
    if (pool->flags & ~GMS_KV_IMAGE_BY_ID) return GMS_ERR_ARG;
    const uint64_t k = pool->block_bytes / gms::kBlockBytes;
    const uint64_t n_slots = (uint64_t)n_sel * pool->n_planes * k;
    if (n_slots >= 0xffffffffull) return GMS_ERR_RANGE;
    if (n_slots && (!d_block_ids || !d_computed || !d_expected || !d_scratch)) return GMS_ERR_NULL;
    gms::VerifyArgs a = {};
    a.computed = d_computed;
    a.expected = d_expected;
    a.n_blocks = n_slots;
    a.seg_count = d_scratch;
    a.n_segments = (uint32_t)((n_slots + gms::kVerifySegBlocks - 1) / gms::kVerifySegBlocks);
    a.out = d_out;
    a.cap = cap;
    a.count = d_count;
    a.kv_ids = d_block_ids;
    a.kv_slots_per_id = (uint32_t)(pool->n_planes * k);
    a.kv_k = (uint32_t)k;
    a.kv_pool_blocks = pool->n_blocks;
    if (a.kv_slots_per_id == 0) a.kv_slots_per_id = 1;  // no planes: there are no slots, nothing is looked up
    GMS_CUDA(gms::launch_verify(a, static_cast<cudaStream_t>(stream)));
    return GMS_OK;
}

int gms_host_image_alloc(uint64_t nbytes, void **host_ptr, void **device_view)
{
    if (!host_ptr || !device_view) return GMS_ERR_NULL;
    *host_ptr = *device_view = nullptr;
    if (nbytes == 0) return GMS_ERR_ARG;
    void *h = nullptr, *d = nullptr;
    cudaError_t e = cudaHostAlloc(&h, nbytes, cudaHostAllocMapped | cudaHostAllocPortable);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        return e == cudaErrorMemoryAllocation ? GMS_ERR_NOMEM : cuda_fail(e);
    }
    e = cudaHostGetDevicePointer(&d, h, 0);
    if (e != cudaSuccess) {
        cudaFreeHost(h);
        return cuda_fail(e);
    }
    *host_ptr = h;
    *device_view = d;
    return GMS_OK;
}

int gms_host_image_free(void *host_ptr)
{
    if (!host_ptr) return GMS_OK;
    GMS_CUDA(cudaFreeHost(host_ptr));
    return GMS_OK;
}

int gms_launch_geometry(uint32_t *grid_ctas, uint32_t *warps_per_cta, uint32_t *smem_bytes)
{
    gms::Geometry g;
    GMS_CUDA(gms::get_geometry(gms::kRestore, &g));
    if (grid_ctas) *grid_ctas = g.grid;
    if (warps_per_cta) *warps_per_cta = g.warps;
    if (smem_bytes) *smem_bytes = g.smem;
    return GMS_OK;
}

uint64_t gms_kernel_launches(void) { return g_launches.load(std::memory_order_relaxed); }

int gms_set_device(int device)
{
    GMS_CUDA(cudaSetDevice(device));
    return GMS_OK;
}

const char *gms_strerror(int status)
{
    switch (status) {
    case GMS_OK: return "ok";
    case GMS_ERR_NULL: return "a required pointer is NULL";
    case GMS_ERR_ALIGN: return "offset, pointer or stride is not 16-byte aligned (or block_bytes is not a multiple of 4096)";
    case GMS_ERR_RANGE: return "range exceeds the image or an index limit";
    case GMS_ERR_OVERLAP: return "destination ranges overlap";
    case GMS_ERR_DUP_ID: return "duplicate tensor_id";
    case GMS_ERR_NOMEM: return "out of memory for the manifest's tables";
    case GMS_ERR_CUDA: return "a CUDA call failed (see gms_last_cuda_error)";
    case GMS_ERR_KIND: return "image pointer does not match image_kind";
    case GMS_ERR_TIMEOUT: return "a bounded device-side wait expired";
    case GMS_ERR_STATE: return "manifest lacks device tables or recorded digests";
    case GMS_ERR_ARG: return "argument out of range";
    case GMS_ERR_IO: return "a file read failed or the file is shorter than the image";
    case GMS_ERR_TOO_LARGE: return "size exceeds the fixed capacity of the no-allocation entry point (GMS_NOALLOC_MAX_BLOCKS)";
    default: return "unknown status";
    }
}

const char *gms_last_cuda_error(void) { return t_cuda_error.c_str(); }

uint32_t gms_version(void) { return 0x00010000u; }

}  // extern "C"
