// gms_restore_fd: storage -> pinned host buffers -> device allocations, pipelined; gms_capture_fd: the way back.
//
// Section 4 (GMS paragraph) has a fresh writer fill a cold service from storage while the process
// itself is being restored; Section 3.1 prices that at S / B_eff and Section 3.3 notes that restoring
// the runtime state leaves storage bandwidth unused.  This file is that leg: the snapshot
// image is never resident as a whole.  A small ring of pinned buffers is filled by a pool of reader
// threads (pread; O_DIRECT where the file system takes it, the page cache otherwise), each filled
// buffer is moved by the copy engine (cudaMemcpyAsync on an internal stream) into one of two device
// buffers, and the restore kernel is launched on the chunks whose sources lie in that window, reading
// device memory and scattering + digesting as usual.  Reading window k+1 overlaps the copy and the
// kernel of window k; a pinned buffer is refilled once its copy has completed, a device buffer once
// the kernel that read it has (CUDA events).  If the device buffers cannot be had, the kernel reads the
// pinned buffers across the host link instead (about 7 % slower on the link).
// All waiting is on the host (condition variables, cudaEventSynchronize); no kernel waits for a flag.
#include <algorithm>
#include <condition_variable>
#include <cerrno>
#include <cstring>
#include <chrono>
#include <deque>
#include <functional>
#include <mutex>
#include <thread>
#include <utility>
#include <vector>

#include <atomic>
#include <fcntl.h>
#include <sys/mman.h>
#include <sys/stat.h>
#include <unistd.h>

#include "../../include/gms.h"
#include "gms_internal.h"

namespace {

class ReaderPool {
  public:
    explicit ReaderPool(uint32_t n)
    {
        for (uint32_t i = 0; i < n; ++i) threads_.emplace_back([this] { run(); });
    }
    ~ReaderPool()
    {
        {
            std::lock_guard<std::mutex> l(mu_);
            stop_ = true;
        }
        cv_.notify_all();
        for (auto &t : threads_) t.join();
    }
    void submit(std::function<void()> f)
    {
        {
            std::lock_guard<std::mutex> l(mu_);
            q_.push_back(std::move(f));
        }
        cv_.notify_one();
    }
    uint32_t size() const { return (uint32_t)threads_.size(); }

  private:
    void run()
    {
        for (;;) {
            std::function<void()> f;
            {
                std::unique_lock<std::mutex> l(mu_);
                cv_.wait(l, [this] { return stop_ || !q_.empty(); });
                if (q_.empty()) return;
                f = std::move(q_.front());
                q_.pop_front();
            }
            f();
        }
    }
    std::mutex mu_;
    std::condition_variable cv_;
    std::deque<std::function<void()>> q_;
    std::vector<std::thread> threads_;
    bool stop_ = false;
};

// completion state of the reads of one window
struct WindowReads {
    std::mutex mu;
    std::condition_variable cv;
    uint32_t pending = 0;
    int error = 0;  // errno of a failed read, or -1 for an unexpected end of file
};

double now_s()
{
    return std::chrono::duration<double>(std::chrono::steady_clock::now().time_since_epoch()).count();
}

}  // namespace

struct gms_pipe {
    uint32_t n_buffers = 0;
    uint64_t buffer_bytes = 0;
    std::vector<void *> host;    // pinned buffers
    std::vector<void *> dview;   // their device-side addresses
    std::vector<cudaEvent_t> done;  // the last reader of pinned buffer b (copy, or kernel when there is no device ring) is finished
    // device ring fed by the copy engine (empty: kernels read the pinned buffers themselves)
    std::vector<void *> dev;
    std::vector<cudaEvent_t> copied;    // device buffer d holds its window (recorded on the copy stream)
    std::vector<cudaEvent_t> consumed;  // the kernel that read device buffer d has finished (caller's stream)
    cudaStream_t copy_stream = nullptr;
    uint64_t dev_uses = 0;              // windows pushed through the device ring so far (across calls)
    bool direct_io = false;             // gms_pipe_direct_io: read with O_DIRECT where the file system allows it
    bool mapped_writes = false;         // gms_pipe_mapped_writes: gms_capture_fd stores through a shared mapping of the file
    ReaderPool *pool = nullptr;
    std::mutex busy;             // one restore at a time per pipe
};

// Device-side staging ring for host images that are moved by the copy engine (gms_restore_staged).
struct gms_stage {
    uint32_t n_buffers = 0;
    uint64_t buffer_bytes = 0;
    std::vector<void *> dev;            // device buffers
    std::vector<cudaEvent_t> copied;    // buffer b holds its window (recorded on the copy stream)
    std::vector<cudaEvent_t> consumed;  // the kernel that read buffer b has finished (recorded on the caller's stream)
    cudaStream_t copy_stream = nullptr;
    uint64_t uses = 0;                  // windows pushed through the ring so far (across calls)
    std::mutex busy;
};

extern "C" {

int gms_stage_create(uint32_t n_buffers, uint64_t buffer_bytes, gms_stage **out)
{
    if (!out) return GMS_ERR_NULL;
    *out = nullptr;
    if (n_buffers < 2 || n_buffers > 64) return GMS_ERR_ARG;
    if (buffer_bytes < (1ull << 20) || (buffer_bytes & 4095u)) return GMS_ERR_ARG;
    gms_stage *st = new (std::nothrow) gms_stage();
    if (!st) return GMS_ERR_NOMEM;
    st->n_buffers = n_buffers;
    st->buffer_bytes = buffer_bytes;
    cudaError_t e = cudaStreamCreateWithFlags(&st->copy_stream, cudaStreamNonBlocking);
    for (uint32_t b = 0; b < n_buffers && e == cudaSuccess; ++b) {
        void *d = nullptr;
        cudaEvent_t a = nullptr, c = nullptr;
        e = cudaMalloc(&d, buffer_bytes);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&a, cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c, cudaEventDisableTiming);
        if (d) st->dev.push_back(d);
        if (a) st->copied.push_back(a);
        if (c) st->consumed.push_back(c);
    }
    if (e != cudaSuccess) {
        const int rc = e == cudaErrorMemoryAllocation ? GMS_ERR_NOMEM : gms::report_cuda_error(e);
        (void)cudaGetLastError();
        for (void *d : st->dev) cudaFree(d);
        for (cudaEvent_t ev : st->copied) cudaEventDestroy(ev);
        for (cudaEvent_t ev : st->consumed) cudaEventDestroy(ev);
        if (st->copy_stream) cudaStreamDestroy(st->copy_stream);
        delete st;
        return rc;
    }
    *out = st;
    return GMS_OK;
}

int gms_stage_destroy(gms_stage *st)
{
    if (!st) return GMS_OK;
    int rc = GMS_OK;
    if (cudaStreamSynchronize(st->copy_stream) != cudaSuccess) rc = GMS_ERR_CUDA;
    for (cudaEvent_t ev : st->consumed)
        if (cudaEventSynchronize(ev) != cudaSuccess) rc = GMS_ERR_CUDA;
    for (void *d : st->dev)
        if (cudaFree(d) != cudaSuccess) rc = GMS_ERR_CUDA;
    for (cudaEvent_t ev : st->copied) cudaEventDestroy(ev);
    for (cudaEvent_t ev : st->consumed) cudaEventDestroy(ev);
    cudaStreamDestroy(st->copy_stream);
    delete st;
    return rc;
}

int gms_restore_staged(const gms_manifest *m, gms_stage *st, const void *host_image, uint64_t *d_block_digests,
                       uint64_t *d_tensor_digests, void *stream)
{
    if (!m || !st) return GMS_ERR_NULL;
    std::lock_guard<std::mutex> one(st->busy);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    std::vector<gms::SrcWindow> windows;
    int rc = gms::manifest_src_windows(m, st->buffer_bytes, &windows);
    if (rc != GMS_OK) return rc;
    if (!windows.empty() && !host_image) return GMS_ERR_NULL;
    if (windows.empty()) {
        gms::SrcWindow none = {0, 0, 0, 0};
        return gms::manifest_launch_window(m, none, st->dev[0], true, d_block_digests, d_tensor_digests, s);
    }
    cudaPointerAttributes at;
    cudaError_t e = cudaPointerGetAttributes(&at, host_image);
    if (e != cudaSuccess) return gms::report_cuda_error(e);
    if (at.type != cudaMemoryTypeHost) return GMS_ERR_KIND;  // must be pinned host memory: the copy engine reads it
    const uint8_t *host = static_cast<const uint8_t *>(host_image);
    for (size_t w = 0; w < windows.size(); ++w) {
        const uint32_t b = (uint32_t)(st->uses % st->n_buffers);
        // copy engine: wait until the kernel that last read this buffer is done, then fill it
        if (st->uses >= st->n_buffers && (e = cudaStreamWaitEvent(st->copy_stream, st->consumed[b], 0)) != cudaSuccess) break;
        const uint64_t len = windows[w].src_hi - windows[w].src_lo;
        if ((e = cudaMemcpyAsync(st->dev[b], host + windows[w].src_lo, len, cudaMemcpyHostToDevice, st->copy_stream)) != cudaSuccess) break;
        if ((e = cudaEventRecord(st->copied[b], st->copy_stream)) != cudaSuccess) break;
        // caller's stream: wait for the window, restore from it, release the buffer
        if ((e = cudaStreamWaitEvent(s, st->copied[b], 0)) != cudaSuccess) break;
        rc = gms::manifest_launch_window(m, windows[w], st->dev[b], w == 0, d_block_digests, d_tensor_digests, s);
        if (rc != GMS_OK) return rc;
        if ((e = cudaEventRecord(st->consumed[b], s)) != cudaSuccess) break;
        ++st->uses;
    }
    return e == cudaSuccess ? GMS_OK : gms::report_cuda_error(e);
}

int gms_pipe_create(uint32_t n_buffers, uint64_t buffer_bytes, uint32_t n_readers, gms_pipe **out)
{
    if (!out) return GMS_ERR_NULL;
    *out = nullptr;
    if (n_buffers < 2 || n_buffers > 64 || n_readers < 1 || n_readers > 256) return GMS_ERR_ARG;
    if (buffer_bytes < (1ull << 20) || (buffer_bytes & 4095u)) return GMS_ERR_ARG;
    gms_pipe *p = new (std::nothrow) gms_pipe();
    if (!p) return GMS_ERR_NOMEM;
    p->n_buffers = n_buffers;
    p->buffer_bytes = buffer_bytes;
    int rc = GMS_OK;
    for (uint32_t b = 0; b < n_buffers && rc == GMS_OK; ++b) {
        void *h = nullptr, *d = nullptr;
        cudaEvent_t ev = nullptr;
        cudaError_t e = cudaHostAlloc(&h, buffer_bytes, cudaHostAllocMapped | cudaHostAllocPortable);
        if (e == cudaSuccess) e = cudaHostGetDevicePointer(&d, h, 0);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
        if (e != cudaSuccess) {
            if (h) cudaFreeHost(h);
            rc = e == cudaErrorMemoryAllocation ? GMS_ERR_NOMEM : gms::report_cuda_error(e);
            (void)cudaGetLastError();
            break;
        }
        p->host.push_back(h);
        p->dview.push_back(d);
        p->done.push_back(ev);
    }
    if (rc == GMS_OK) {
        p->pool = new (std::nothrow) ReaderPool(n_readers);
        if (!p->pool) rc = GMS_ERR_NOMEM;
    }
    if (rc == GMS_OK) {  // two device buffers for the copy engine to fill; without them the mapped path is used
        cudaError_t e = cudaStreamCreateWithFlags(&p->copy_stream, cudaStreamNonBlocking);
        for (uint32_t d = 0; d < 2 && e == cudaSuccess; ++d) {
            void *buf = nullptr;
            cudaEvent_t a = nullptr, c = nullptr;
            e = cudaMalloc(&buf, buffer_bytes);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&a, cudaEventDisableTiming);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c, cudaEventDisableTiming);
            if (buf) p->dev.push_back(buf);
            if (a) p->copied.push_back(a);
            if (c) p->consumed.push_back(c);
        }
        if (e != cudaSuccess) {
            (void)cudaGetLastError();
            for (void *buf : p->dev) cudaFree(buf);
            for (cudaEvent_t ev : p->copied) cudaEventDestroy(ev);
            for (cudaEvent_t ev : p->consumed) cudaEventDestroy(ev);
            p->dev.clear();
            p->copied.clear();
            p->consumed.clear();
            if (e != cudaErrorMemoryAllocation) rc = gms::report_cuda_error(e);
        }
    }
    if (rc != GMS_OK) {
        for (void *h : p->host) cudaFreeHost(h);
        for (cudaEvent_t ev : p->done) cudaEventDestroy(ev);
        if (p->copy_stream) cudaStreamDestroy(p->copy_stream);
        delete p->pool;
        delete p;
        return rc;
    }
    *out = p;
    return GMS_OK;
}

int gms_pipe_direct_io(gms_pipe *p, int enable)
{
    if (!p) return GMS_ERR_NULL;
    std::lock_guard<std::mutex> one(p->busy);
    p->direct_io = enable != 0;
    return GMS_OK;
}

int gms_pipe_mapped_writes(gms_pipe *p, int enable)
{
    if (!p) return GMS_ERR_NULL;
    std::lock_guard<std::mutex> one(p->busy);
    p->mapped_writes = enable != 0;
    return GMS_OK;
}

int gms_pipe_destroy(gms_pipe *p)
{
    if (!p) return GMS_OK;
    delete p->pool;  // joins the readers
    int rc = GMS_OK;
    if (p->copy_stream && cudaStreamSynchronize(p->copy_stream) != cudaSuccess) rc = GMS_ERR_CUDA;
    for (cudaEvent_t ev : p->consumed)
        if (cudaEventSynchronize(ev) != cudaSuccess) rc = GMS_ERR_CUDA;
    for (void *buf : p->dev)
        if (cudaFree(buf) != cudaSuccess) rc = GMS_ERR_CUDA;
    for (cudaEvent_t ev : p->copied) cudaEventDestroy(ev);
    for (cudaEvent_t ev : p->consumed) cudaEventDestroy(ev);
    if (p->copy_stream) cudaStreamDestroy(p->copy_stream);
    for (cudaEvent_t ev : p->done)
        if (cudaEventDestroy(ev) != cudaSuccess) rc = GMS_ERR_CUDA;
    for (void *h : p->host)
        if (cudaFreeHost(h) != cudaSuccess) rc = GMS_ERR_CUDA;
    delete p;
    return rc;
}

int gms_restore_fd(const gms_manifest *m, gms_pipe *p, int fd, uint64_t file_offset, uint64_t *d_block_digests,
                   uint64_t *d_tensor_digests, void *stream, gms_pipe_stats *stats)
{
    if (!m || !p) return GMS_ERR_NULL;
    if (fd < 0) return GMS_ERR_ARG;
    std::lock_guard<std::mutex> one(p->busy);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    std::vector<gms::SrcWindow> windows;
    // a window is read from the 4 KiB boundary below its first byte (so that direct reads stay aligned): leave room
    int rc = gms::manifest_src_windows(m, p->buffer_bytes - 4096, &windows);
    if (rc != GMS_OK) return rc;
    const double t_start = now_s();
    gms_pipe_stats st = {};
    st.windows = windows.size();

    if (windows.empty()) {  // nothing to move: still clear the accumulators
        gms::SrcWindow none = {0, 0, 0, 0};
        rc = gms::manifest_launch_window(m, none, p->dview[0], true, d_block_digests, d_tensor_digests, s);
    }

    std::vector<WindowReads> reads(windows.size());
    const uint32_t n_readers = p->pool->size();
    size_t next_read = 0, next_launch = 0;
    int io_error = 0;
    const bool staged = !p->dev.empty();
    // On request (gms_pipe_direct_io): a second descriptor on the same file that bypasses the page cache, where the
    // file system allows it (where it does not, the open or the first read fails and the ordinary descriptor is used).
    // Direct reads need 4 KiB-aligned file offsets, addresses and lengths, so every window is read from the 4 KiB
    // boundary below its first byte and used from `shift` bytes into its buffer (the kernel's sources must stay
    // 16-byte aligned, which they do when file_offset is a multiple of 16; otherwise nothing is shifted and only
    // slices that happen to be aligned go direct).
    char proc_path[64];
    snprintf(proc_path, sizeof proc_path, "/proc/self/fd/%d", fd);
    const int dfd = p->direct_io ? open(proc_path, O_RDONLY | O_DIRECT | O_CLOEXEC) : -1;
    std::atomic<bool> direct_ok{dfd >= 0};
    const bool shifted = dfd >= 0 && (file_offset & 15u) == 0;
    std::vector<uint32_t> shifts(windows.size(), 0);
    while (rc == GMS_OK && next_launch < windows.size()) {
        // start reads as far ahead as the ring allows
        while (next_read < windows.size() && next_read < next_launch + p->n_buffers) {
            const uint32_t b = (uint32_t)(next_read % p->n_buffers);
            if (next_read >= p->n_buffers) {  // the kernel that read this buffer last must be done with it
                const double t0 = now_s();
                cudaError_t e = cudaEventSynchronize(p->done[b]);
                st.wait_gpu_seconds += now_s() - t0;
                if (e != cudaSuccess) {
                    rc = gms::report_cuda_error(e);
                    break;
                }
            }
            const gms::SrcWindow &w = windows[next_read];
            WindowReads &wr = reads[next_read];
            const uint64_t len = w.src_hi - w.src_lo;
            if (next_read + 1 < windows.size())  // tell the kernel which bytes come next (a hint; errors do not matter)
                (void)posix_fadvise(fd, (off_t)(file_offset + windows[next_read + 1].src_lo),
                                    (off_t)(windows[next_read + 1].src_hi - windows[next_read + 1].src_lo), POSIX_FADV_WILLNEED);
            const uint64_t shift = shifted ? ((file_offset + w.src_lo) & 4095u) : 0;
            shifts[next_read] = (uint32_t)shift;
            const uint64_t span = len + shift;  // bytes read into the buffer, from its start
            // slices are multiples of 1 MiB so that readers do not share pages
            uint64_t slice = (span + n_readers - 1) / n_readers;
            slice = (slice + (1u << 20) - 1) & ~((uint64_t)(1u << 20) - 1);
            const uint32_t n_slices = (uint32_t)((span + slice - 1) / slice);
            wr.pending = n_slices;
            uint8_t *base = static_cast<uint8_t *>(p->host[b]);
            for (uint32_t k = 0; k < n_slices; ++k) {
                const uint64_t lo = (uint64_t)k * slice, n = std::min<uint64_t>(slice, span - lo);
                const uint64_t foff = file_offset + w.src_lo - shift + lo;
                p->pool->submit([fd, dfd, &direct_ok, base, lo, n, foff, &wr] {
                    uint64_t got = 0;
                    int err = 0;
                    // the 4 KiB-aligned body of the slice through the direct descriptor, if it still works
                    const uint64_t body = n & ~(uint64_t)4095;
                    if (body && direct_ok.load(std::memory_order_relaxed) && (foff & 4095u) == 0 &&
                        (reinterpret_cast<uint64_t>(base + lo) & 4095u) == 0) {
                        while (got < body) {
                            const ssize_t r = pread(dfd, base + lo + got, body - got, (off_t)(foff + got));
                            if (r < 0 && errno == EINTR) continue;
                            if (r <= 0 || (r & 4095)) {  // refused, short or ragged: the ordinary descriptor takes over
                                if (r < 0) direct_ok.store(false, std::memory_order_relaxed);
                                if (r > 0) got += (uint64_t)r;
                                break;
                            }
                            got += (uint64_t)r;
                        }
                    }
                    while (got < n) {
                        const ssize_t r = pread(fd, base + lo + got, n - got, (off_t)(foff + got));
                        if (r < 0) {
                            if (errno == EINTR) continue;
                            err = errno ? errno : -1;
                            break;
                        }
                        if (r == 0) {
                            err = -1;  // file shorter than the image
                            break;
                        }
                        got += (uint64_t)r;
                    }
                    std::lock_guard<std::mutex> l(wr.mu);
                    if (err && !wr.error) wr.error = err;
                    if (--wr.pending == 0) wr.cv.notify_all();
                });
            }
            st.bytes_read += len;
            ++next_read;
        }
        if (rc != GMS_OK) break;
        // wait for the window to be launched next, then launch it
        {
            WindowReads &wr = reads[next_launch];
            const double t0 = now_s();
            std::unique_lock<std::mutex> l(wr.mu);
            wr.cv.wait(l, [&wr] { return wr.pending == 0; });
            st.wait_read_seconds += now_s() - t0;
            if (wr.error) {
                io_error = wr.error;
                break;
            }
        }
        const uint32_t b = (uint32_t)(next_launch % p->n_buffers);
        if (staged) {
            // copy engine: pinned buffer b -> device buffer d (once the kernel that last read d is done), then the
            // kernel on the caller's stream reads d; the pinned buffer is free again when the copy has completed
            const uint32_t d = (uint32_t)(p->dev_uses % p->dev.size());
            const gms::SrcWindow &w = windows[next_launch];
            cudaError_t e = cudaSuccess;
            if (p->dev_uses >= p->dev.size()) e = cudaStreamWaitEvent(p->copy_stream, p->consumed[d], 0);
            if (e == cudaSuccess)
                e = cudaMemcpyAsync(p->dev[d], static_cast<const uint8_t *>(p->host[b]) + shifts[next_launch], w.src_hi - w.src_lo,
                                    cudaMemcpyHostToDevice, p->copy_stream);
            if (e == cudaSuccess) e = cudaEventRecord(p->copied[d], p->copy_stream);
            if (e == cudaSuccess) e = cudaEventRecord(p->done[b], p->copy_stream);
            if (e == cudaSuccess) e = cudaStreamWaitEvent(s, p->copied[d], 0);
            if (e != cudaSuccess) {
                rc = gms::report_cuda_error(e);
                break;
            }
            rc = gms::manifest_launch_window(m, w, p->dev[d], next_launch == 0, d_block_digests, d_tensor_digests, s);
            if (rc == GMS_OK && (e = cudaEventRecord(p->consumed[d], s)) != cudaSuccess) rc = gms::report_cuda_error(e);
            ++p->dev_uses;
        } else {
            rc = gms::manifest_launch_window(m, windows[next_launch], static_cast<const uint8_t *>(p->dview[b]) + shifts[next_launch],
                                             next_launch == 0, d_block_digests, d_tensor_digests, s);
            if (rc == GMS_OK) {
                cudaError_t e = cudaEventRecord(p->done[b], s);
                if (e != cudaSuccess) rc = gms::report_cuda_error(e);
            }
        }
        ++next_launch;
    }
    // drain: reads still in flight must not outlive this call (they write into the pipe's buffers and use `reads`)
    for (size_t w = 0; w < next_read; ++w) {
        std::unique_lock<std::mutex> l(reads[w].mu);
        reads[w].cv.wait(l, [&] { return reads[w].pending == 0; });
    }
    if (dfd >= 0) close(dfd);
    cudaError_t e = staged ? cudaStreamSynchronize(p->copy_stream) : cudaSuccess;
    if (e != cudaSuccess && rc == GMS_OK) rc = gms::report_cuda_error(e);
    e = cudaStreamSynchronize(s);
    if (e != cudaSuccess && rc == GMS_OK) rc = gms::report_cuda_error(e);
    st.direct_io = dfd >= 0 && direct_ok.load() ? 1u : 0u;
    st.copy_engine = staged ? 1u : 0u;
    st.total_seconds = now_s() - t_start;
    if (stats) *stats = st;
    if (io_error) return GMS_ERR_IO;
    return rc;
}

// The other direction: device allocations -> pinned buffers -> file (Section 3.1: step 3 stages device state into
// host memory, step 4 serialises it to durable storage).  The capture kernel gathers one window of the image at a
// time straight into a pinned buffer (kernel-issued bulk stores across the host link run at the rate of the copy
// engine in this direction, so there is no device-side staging), and the pipe's threads write the window's tensor
// ranges to the file with pwrite while the kernel fills the next buffer.  Only bytes that belong to a tensor are
// written: what the file holds between two tensors' ranges stays as it was.
int gms_capture_fd(const gms_manifest *m, gms_pipe *p, int fd, uint64_t file_offset, uint64_t *d_block_digests,
                   uint64_t *d_tensor_digests, void *stream, gms_pipe_stats *stats)
{
    if (!m || !p) return GMS_ERR_NULL;
    if (fd < 0) return GMS_ERR_ARG;
    std::lock_guard<std::mutex> one(p->busy);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    std::vector<std::pair<uint64_t, uint64_t>> ranges;  // image ranges of the tensors, ascending
    int rc = gms::manifest_sorted_sources(m, &ranges);
    if (rc != GMS_OK) return rc;
    std::vector<gms::SrcWindow> windows;
    rc = gms::manifest_src_windows(m, p->buffer_bytes, &windows);
    if (rc != GMS_OK) return rc;
    const double t_start = now_s();
    gms_pipe_stats st = {};
    st.windows = windows.size();
    if (windows.empty()) {  // nothing to move: still clear the accumulators
        gms::SrcWindow none = {0, 0, 0, 0};
        rc = gms::manifest_launch_window(m, none, p->dview[0], true, d_block_digests, d_tensor_digests, s, true);
    }

    // On request (gms_pipe_mapped_writes): the writers copy into a shared mapping of the file instead of calling pwrite.
    // Buffered writes to one file are serialised by the kernel (one writer holds the file's lock at a time), stores
    // into a mapping are not, so for a file that lives in the page cache this is the difference between one core's
    // copy rate and all of them.  Only for a regular file that already spans the image (a store beyond the end of
    // the file would raise SIGBUS) on a descriptor that allows a shared writable mapping; pwrite otherwise.
    uint8_t *map = nullptr;
    uint64_t map_lo = 0, map_len = 0;
    if (p->mapped_writes && !windows.empty()) {
        struct stat sb;
        const uint64_t lo = file_offset + windows.front().src_lo, hi = file_offset + windows.back().src_hi;
        if (fstat(fd, &sb) == 0 && S_ISREG(sb.st_mode) && (uint64_t)sb.st_size >= hi) {
            map_lo = lo & ~(uint64_t)4095;
            map_len = hi - map_lo;
            void *a = mmap(nullptr, map_len, PROT_READ | PROT_WRITE, MAP_SHARED, fd, (off_t)map_lo);
            if (a != MAP_FAILED) map = static_cast<uint8_t *>(a);
        }
    }
    st.mapped_io = map ? 1u : 0u;

    struct Piece {
        uint64_t buf_off, file_off, n;
    };
    std::vector<WindowReads> writes(windows.size());  // completion state of each window's writes
    const uint32_t n_writers = p->pool->size();
    size_t next_launch = 0, next_write = 0, ri = 0;  // ri: first tensor range that reaches into the window to write
    int io_error = 0;
    auto wait_written = [&](size_t w) {
        const double t0 = now_s();
        std::unique_lock<std::mutex> l(writes[w].mu);
        writes[w].cv.wait(l, [&] { return writes[w].pending == 0; });
        st.wait_read_seconds += now_s() - t0;
        if (writes[w].error && !io_error) io_error = writes[w].error;
    };
    while (rc == GMS_OK && !io_error && next_write < windows.size()) {
        // gather as far ahead as the ring allows: a buffer is free once the window it held has been written out
        while (next_launch < windows.size() && next_launch < next_write + p->n_buffers) {
            if (next_launch >= p->n_buffers) wait_written(next_launch - p->n_buffers);
            if (io_error) break;
            const uint32_t b = (uint32_t)(next_launch % p->n_buffers);
            rc = gms::manifest_launch_window(m, windows[next_launch], p->dview[b], next_launch == 0, d_block_digests,
                                             d_tensor_digests, s, true);
            if (rc != GMS_OK) break;
            cudaError_t e = cudaEventRecord(p->done[b], s);
            if (e != cudaSuccess) {
                rc = gms::report_cuda_error(e);
                break;
            }
            ++next_launch;
        }
        if (rc != GMS_OK || io_error) break;
        // the window to write next: wait for its kernel, then hand its tensor ranges to the writers
        const gms::SrcWindow &w = windows[next_write];
        const uint32_t b = (uint32_t)(next_write % p->n_buffers);
        {
            const double t0 = now_s();
            cudaError_t e = cudaEventSynchronize(p->done[b]);
            st.wait_gpu_seconds += now_s() - t0;
            if (e != cudaSuccess) {
                rc = gms::report_cuda_error(e);
                break;
            }
        }
        // the tensor bytes inside [src_lo, src_hi), adjacent ranges merged, cut into jobs of about a writer's share
        uint64_t slice = (w.src_hi - w.src_lo + n_writers - 1) / n_writers;
        slice = std::max<uint64_t>((slice + (1u << 20) - 1) & ~((uint64_t)(1u << 20) - 1), 1u << 20);
        std::vector<std::vector<Piece>> jobs(1);
        uint64_t job_bytes = 0;
        while (ri < ranges.size() && ranges[ri].first + ranges[ri].second <= w.src_lo) ++ri;
        for (size_t k = ri; k < ranges.size() && ranges[k].first < w.src_hi; ++k) {
            uint64_t lo = std::max(ranges[k].first, w.src_lo);
            const uint64_t hi = std::min(ranges[k].first + ranges[k].second, w.src_hi);
            while (lo < hi) {
                const uint64_t n = std::min(hi - lo, slice - job_bytes);
                std::vector<Piece> &job = jobs.back();
                if (!job.empty() && job.back().buf_off + job.back().n == lo - w.src_lo)
                    job.back().n += n;  // continues the piece before it
                else
                    job.push_back({lo - w.src_lo, file_offset + lo, n});
                lo += n;
                job_bytes += n;
                st.bytes_read += n;
                if (job_bytes == slice) jobs.emplace_back(), job_bytes = 0;
            }
        }
        if (jobs.back().empty()) jobs.pop_back();
        WindowReads &wr = writes[next_write];
        wr.pending = (uint32_t)jobs.size();
        const uint8_t *base = static_cast<const uint8_t *>(p->host[b]);
        for (std::vector<Piece> &job : jobs)
            p->pool->submit([fd, base, map, map_lo, &wr, pieces = std::move(job)] {
                int err = 0;
                for (const Piece &pc : pieces) {
                    if (map) {
                        uint8_t *to = map + (pc.file_off - map_lo);
#ifdef MADV_POPULATE_WRITE
                        // map the piece's pages in one call instead of one fault per page (a hint: errors do not matter)
                        if (pc.n >= (1u << 16)) {
                            uint8_t *lo = reinterpret_cast<uint8_t *>(reinterpret_cast<uint64_t>(to) & ~(uint64_t)4095);
                            (void)madvise(lo, (size_t)(to + pc.n - lo), MADV_POPULATE_WRITE);
                        }
#endif
                        memcpy(to, base + pc.buf_off, pc.n);
                        continue;
                    }
                    uint64_t put = 0;
                    while (put < pc.n && !err) {
                        const ssize_t r = pwrite(fd, base + pc.buf_off + put, pc.n - put, (off_t)(pc.file_off + put));
                        if (r < 0 && errno == EINTR) continue;
                        if (r <= 0)
                            err = (r < 0 && errno) ? errno : -1;
                        else
                            put += (uint64_t)r;
                    }
                    if (err) break;
                }
                std::lock_guard<std::mutex> l(wr.mu);
                if (err && !wr.error) wr.error = err;
                if (--wr.pending == 0) wr.cv.notify_all();
            });
        ++next_write;
    }
    // drain: writers use the pipe's buffers and `writes`, kernels write the buffers: neither may outlive this call
    for (size_t w = 0; w < next_write; ++w) wait_written(w);
    if (map) munmap(map, map_len);
    cudaError_t e = cudaStreamSynchronize(s);
    if (e != cudaSuccess && rc == GMS_OK) rc = gms::report_cuda_error(e);
    st.total_seconds = now_s() - t_start;
    if (stats) *stats = st;
    if (io_error) return GMS_ERR_IO;
    return rc;
}

}  // extern "C"
