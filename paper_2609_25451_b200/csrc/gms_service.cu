// gms_service_*: the substrate under the destinations -- service-owned device allocations with the
// paper's ownership protocol, in one process.
//
// Section 4 (GMS paragraph): the service creates physical allocations with cuMemCreate and keeps
// the number of VMM calls down by suballocating, first fit, out of 2 GiB slabs, giving any single
// allocation above 2 GiB a slab of its own, so mapping and permission set-up happen per slab, not
// per tensor.  Section 3.2 / Figure (ownership protocol): EMPTY -> RW (one
// writer populates) -> COMMITTED (immutable, no readers) <-> RO (n >= 1 readers); a writer that
// gives up before commit discards the state; write access is available again once the last
// reader has left; read-only access is enforced with cuMemSetAccess.
//
// What is here: slabs created / reserved / mapped with the CUDA virtual-memory-management driver
// calls (looked up through cudaGetDriverEntryPoint, so the library does not link libcuda), a
// first-fit free list per slab, and the state machine.  Commit flips every slab to read-only;
// re-acquiring write access flips it back and keeps contents and addresses (repair in place).
// Across processes (Section 4, GMS paragraph: the service keeps the creator handles and hands clients file
// descriptors over Unix sockets; clients import them, map them and set their own access): a service created
// with GMS_SERVICE_SHAREABLE makes its slabs exportable, gms_service_export_fd turns a slab into a descriptor,
// and gms_import_* is the client's side -- import, reserve (at the service's address if asked), map, read-only
// or writable.  The socket and the messages on it belong to the processes that use this, not to the library.
// A dry-run backend (no CUDA call, addresses from a counter) lets the bookkeeping be tested without
// a GPU.  Nothing in this file ever writes through a read-only mapping.
#include <algorithm>
#include <mutex>
#include <new>
#include <vector>

#include <cuda.h>

#include "../../include/gms.h"
#include "gms_internal.h"

namespace {

struct Driver {
    CUresult (*memCreate)(CUmemGenericAllocationHandle *, size_t, const CUmemAllocationProp *, unsigned long long) = nullptr;
    CUresult (*memRelease)(CUmemGenericAllocationHandle) = nullptr;
    CUresult (*memAddressReserve)(CUdeviceptr *, size_t, size_t, CUdeviceptr, unsigned long long) = nullptr;
    CUresult (*memAddressFree)(CUdeviceptr, size_t) = nullptr;
    CUresult (*memMap)(CUdeviceptr, size_t, size_t, CUmemGenericAllocationHandle, unsigned long long) = nullptr;
    CUresult (*memUnmap)(CUdeviceptr, size_t) = nullptr;
    CUresult (*memSetAccess)(CUdeviceptr, size_t, const CUmemAccessDesc *, size_t) = nullptr;
    CUresult (*memGetAccess)(unsigned long long *, const CUmemLocation *, CUdeviceptr) = nullptr;
    CUresult (*memGetAllocationGranularity)(size_t *, const CUmemAllocationProp *, CUmemAllocationGranularity_flags) = nullptr;
    CUresult (*memExportToShareableHandle)(void *, CUmemGenericAllocationHandle, CUmemAllocationHandleType, unsigned long long) = nullptr;
    CUresult (*memImportFromShareableHandle)(CUmemGenericAllocationHandle *, void *, CUmemAllocationHandleType) = nullptr;
    bool ok = false;
};

template <class F>
bool lookup(const char *name, F *fn)
{
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint(name, &p, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess || !p) {
        (void)cudaGetLastError();
        return false;
    }
    *fn = reinterpret_cast<F>(p);
    return true;
}

Driver *driver()
{
    static Driver d;
    static std::once_flag once;
    std::call_once(once, [] {
        d.ok = lookup("cuMemCreate", &d.memCreate) && lookup("cuMemRelease", &d.memRelease) &&
               lookup("cuMemAddressReserve", &d.memAddressReserve) && lookup("cuMemAddressFree", &d.memAddressFree) &&
               lookup("cuMemMap", &d.memMap) && lookup("cuMemUnmap", &d.memUnmap) && lookup("cuMemSetAccess", &d.memSetAccess) &&
               lookup("cuMemGetAccess", &d.memGetAccess) &&
               lookup("cuMemGetAllocationGranularity", &d.memGetAllocationGranularity) &&
               lookup("cuMemExportToShareableHandle", &d.memExportToShareableHandle) &&
               lookup("cuMemImportFromShareableHandle", &d.memImportFromShareableHandle);
    });
    return &d;
}

struct FreeRun {
    uint64_t off, len;
};

struct Slab {
    uint64_t va = 0, size = 0;
    CUmemGenericAllocationHandle handle = 0;
    bool dedicated = false;          // holds one allocation larger than the slab size
    std::vector<FreeRun> free_runs;  // sorted by offset, coalesced
    uint64_t used = 0;
};

constexpr uint64_t kAllocAlign = 256;

}  // namespace

struct gms_service {
    std::mutex mu;
    int device = 0;
    bool dry_run = false;
    bool shareable = false;  // slabs can be exported as file descriptors
    uint64_t slab_bytes = 0, granularity = 2ull << 20;
    uint64_t fake_next_va = 0x700000000000ull;
    uint32_t state = GMS_STATE_EMPTY, readers = 0;
    bool attached = true;  // slabs are mapped into the address space (false between detach and reattach)
    bool backed = true;    // slabs have physical memory (false between release_pages and back_pages)
    std::vector<Slab> slabs;
};

namespace {

CUmemAllocationProp slab_prop(int device, bool shareable)
{
    CUmemAllocationProp prop = {};
    prop.type = CU_MEM_ALLOCATION_TYPE_PINNED;
    prop.location.type = CU_MEM_LOCATION_TYPE_DEVICE;
    prop.location.id = device;
    if (shareable) prop.requestedHandleTypes = CU_MEM_HANDLE_TYPE_POSIX_FILE_DESCRIPTOR;
    return prop;
}

int set_access(gms_service *s, const Slab &slab, bool writable)
{
    if (s->dry_run) return GMS_OK;
    CUmemAccessDesc desc = {};
    desc.location.type = CU_MEM_LOCATION_TYPE_DEVICE;
    desc.location.id = s->device;
    desc.flags = writable ? CU_MEM_ACCESS_FLAGS_PROT_READWRITE : CU_MEM_ACCESS_FLAGS_PROT_READ;
    return driver()->memSetAccess((CUdeviceptr)slab.va, slab.size, &desc, 1) == CUDA_SUCCESS ? GMS_OK : GMS_ERR_CUDA;
}

int new_slab(gms_service *s, uint64_t size, bool dedicated, Slab *out)
{
    Slab slab;
    slab.size = (size + s->granularity - 1) / s->granularity * s->granularity;
    slab.dedicated = dedicated;
    if (s->dry_run) {
        slab.va = s->fake_next_va;
        s->fake_next_va += slab.size + (1ull << 30);
    } else {
        Driver *d = driver();
        const CUmemAllocationProp prop = slab_prop(s->device, s->shareable);
        CUresult r = d->memCreate(&slab.handle, slab.size, &prop, 0);
        if (r != CUDA_SUCCESS) return r == CUDA_ERROR_OUT_OF_MEMORY ? GMS_ERR_NOMEM : GMS_ERR_CUDA;
        CUdeviceptr va = 0;
        if (d->memAddressReserve(&va, slab.size, 0, 0, 0) != CUDA_SUCCESS) {
            d->memRelease(slab.handle);
            return GMS_ERR_CUDA;
        }
        if (d->memMap(va, slab.size, 0, slab.handle, 0) != CUDA_SUCCESS) {
            d->memAddressFree(va, slab.size);
            d->memRelease(slab.handle);
            return GMS_ERR_CUDA;
        }
        slab.va = (uint64_t)va;
        if (set_access(s, slab, true) != GMS_OK) {
            d->memUnmap(va, slab.size);
            d->memAddressFree(va, slab.size);
            d->memRelease(slab.handle);
            return GMS_ERR_CUDA;
        }
    }
    slab.free_runs.push_back({0, slab.size});
    *out = slab;
    return GMS_OK;
}

void drop_slab(gms_service *s, Slab &slab)
{
    if (!s->dry_run && slab.va) {
        Driver *d = driver();
        if (s->attached && s->backed) d->memUnmap((CUdeviceptr)slab.va, slab.size);
        d->memAddressFree((CUdeviceptr)slab.va, slab.size);
        if (s->backed) d->memRelease(slab.handle);
    }
    slab.va = 0;
}

// Maps the slab's physical memory at its reserved address again, with the given access.
int map_slab(gms_service *s, Slab &slab, bool writable)
{
    if (s->dry_run) return GMS_OK;
    if (driver()->memMap((CUdeviceptr)slab.va, slab.size, 0, slab.handle, 0) != CUDA_SUCCESS) return GMS_ERR_CUDA;
    return set_access(s, slab, writable);
}

// first fit inside one slab
bool carve(Slab &slab, uint64_t need, uint64_t *off)
{
    for (size_t i = 0; i < slab.free_runs.size(); ++i) {
        FreeRun &r = slab.free_runs[i];
        if (r.len >= need) {
            *off = r.off;
            r.off += need;
            r.len -= need;
            if (r.len == 0) slab.free_runs.erase(slab.free_runs.begin() + (long)i);
            slab.used += need;
            return true;
        }
    }
    return false;
}

int quiesce(gms_service *s)
{
    if (s->dry_run) return GMS_OK;
    cudaError_t e = cudaDeviceSynchronize();  // no copy may be in flight while permissions change
    return e == cudaSuccess ? GMS_OK : gms::report_cuda_error(e);
}

void discard_all(gms_service *s)
{
    for (Slab &slab : s->slabs) drop_slab(s, slab);
    s->slabs.clear();
}

}  // namespace

extern "C" {

int gms_service_create(uint64_t slab_bytes, uint32_t flags, gms_service **out)
{
    if (!out) return GMS_ERR_NULL;
    *out = nullptr;
    if (flags & ~(GMS_SERVICE_DRY_RUN | GMS_SERVICE_SHAREABLE)) return GMS_ERR_ARG;
    gms_service *s = new (std::nothrow) gms_service();
    if (!s) return GMS_ERR_NOMEM;
    s->dry_run = (flags & GMS_SERVICE_DRY_RUN) != 0;
    s->shareable = (flags & GMS_SERVICE_SHAREABLE) != 0;
    if (!s->dry_run) {
        cudaError_t e = cudaFree(nullptr);  // make sure the primary context exists and is current
        if (e == cudaSuccess) e = cudaGetDevice(&s->device);
        if (e != cudaSuccess) {
            delete s;
            return gms::report_cuda_error(e);
        }
        if (!driver()->ok) {
            delete s;
            return GMS_ERR_CUDA;
        }
        const CUmemAllocationProp prop = slab_prop(s->device, s->shareable);
        size_t g = 0;
        if (driver()->memGetAllocationGranularity(&g, &prop, CU_MEM_ALLOC_GRANULARITY_RECOMMENDED) != CUDA_SUCCESS || g == 0) {
            delete s;
            return GMS_ERR_CUDA;
        }
        s->granularity = g;
    }
    s->slab_bytes = slab_bytes ? slab_bytes : (2ull << 30);
    s->slab_bytes = (s->slab_bytes + s->granularity - 1) / s->granularity * s->granularity;
    *out = s;
    return GMS_OK;
}

int gms_service_destroy(gms_service *s)
{
    if (!s) return GMS_OK;
    int rc = quiesce(s);
    discard_all(s);
    delete s;
    return rc;
}

int gms_service_acquire_rw(gms_service *s)
{
    if (!s) return GMS_ERR_NULL;
    std::lock_guard<std::mutex> l(s->mu);
    if (s->state == GMS_STATE_EMPTY) {
        s->state = GMS_STATE_RW;
        return GMS_OK;
    }
    if (s->state != GMS_STATE_COMMITTED || !s->attached) return GMS_ERR_STATE;  // a writer or readers hold it, or it is detached
    int rc = quiesce(s);
    for (Slab &slab : s->slabs)
        if (rc == GMS_OK) rc = set_access(s, slab, true);
    if (rc != GMS_OK) return rc;
    s->state = GMS_STATE_RW;
    return GMS_OK;
}

int gms_service_alloc(gms_service *s, uint64_t nbytes, void **dptr)
{
    if (!s || !dptr) return GMS_ERR_NULL;
    *dptr = nullptr;
    std::lock_guard<std::mutex> l(s->mu);
    if (s->state != GMS_STATE_RW || !s->backed) return GMS_ERR_STATE;
    if (nbytes == 0 || nbytes > (1ull << 46)) return GMS_ERR_ARG;
    const uint64_t need = (nbytes + kAllocAlign - 1) / kAllocAlign * kAllocAlign;
    uint64_t off = 0;
    if (need <= s->slab_bytes) {
        for (Slab &slab : s->slabs)
            if (!slab.dedicated && carve(slab, need, &off)) {
                *dptr = reinterpret_cast<void *>(slab.va + off);
                return GMS_OK;
            }
    }
    Slab slab;
    const bool dedicated = need > s->slab_bytes;
    int rc = new_slab(s, dedicated ? need : s->slab_bytes, dedicated, &slab);
    if (rc != GMS_OK) return rc;
    carve(slab, need, &off);
    *dptr = reinterpret_cast<void *>(slab.va + off);
    try {
        s->slabs.push_back(slab);
    } catch (const std::bad_alloc &) {
        drop_slab(s, slab);
        *dptr = nullptr;
        return GMS_ERR_NOMEM;
    }
    return GMS_OK;
}

int gms_service_commit(gms_service *s)
{
    if (!s) return GMS_ERR_NULL;
    std::lock_guard<std::mutex> l(s->mu);
    if (s->state != GMS_STATE_RW || !s->backed) return GMS_ERR_STATE;
    int rc = quiesce(s);
    for (Slab &slab : s->slabs)
        if (rc == GMS_OK) rc = set_access(s, slab, false);
    if (rc != GMS_OK) return rc;
    s->state = GMS_STATE_COMMITTED;
    return GMS_OK;
}

int gms_service_abort(gms_service *s)
{
    if (!s) return GMS_ERR_NULL;
    std::lock_guard<std::mutex> l(s->mu);
    if (s->state != GMS_STATE_RW) return GMS_ERR_STATE;
    int rc = quiesce(s);
    discard_all(s);
    s->state = GMS_STATE_EMPTY;
    s->backed = true;
    return rc;
}

int gms_service_detach(gms_service *s)
{
    if (!s) return GMS_ERR_NULL;
    std::lock_guard<std::mutex> l(s->mu);
    if (s->state != GMS_STATE_COMMITTED || !s->attached) return GMS_ERR_STATE;
    int rc = quiesce(s);
    if (rc != GMS_OK) return rc;
    if (!s->dry_run)
        for (Slab &slab : s->slabs)
            if (driver()->memUnmap((CUdeviceptr)slab.va, slab.size) != CUDA_SUCCESS) rc = GMS_ERR_CUDA;
    s->attached = false;
    return rc;
}

int gms_service_reattach(gms_service *s)
{
    if (!s) return GMS_ERR_NULL;
    std::lock_guard<std::mutex> l(s->mu);
    if (s->state != GMS_STATE_COMMITTED || s->attached) return GMS_ERR_STATE;
    int rc = GMS_OK;
    for (Slab &slab : s->slabs)
        if (rc == GMS_OK) rc = map_slab(s, slab, false);  // committed state comes back read-only, at the same addresses
    if (rc != GMS_OK) return rc;
    s->attached = true;
    return GMS_OK;
}

int gms_service_release_pages(gms_service *s)
{
    if (!s) return GMS_ERR_NULL;
    std::lock_guard<std::mutex> l(s->mu);
    if (s->state != GMS_STATE_RW || !s->backed) return GMS_ERR_STATE;
    int rc = quiesce(s);
    if (rc != GMS_OK) return rc;
    if (!s->dry_run)
        for (Slab &slab : s->slabs) {
            if (driver()->memUnmap((CUdeviceptr)slab.va, slab.size) != CUDA_SUCCESS) rc = GMS_ERR_CUDA;
            if (driver()->memRelease(slab.handle) != CUDA_SUCCESS) rc = GMS_ERR_CUDA;
            slab.handle = 0;
        }
    s->backed = false;
    return rc;
}

int gms_service_back_pages(gms_service *s)
{
    if (!s) return GMS_ERR_NULL;
    std::lock_guard<std::mutex> l(s->mu);
    if (s->state != GMS_STATE_RW || s->backed) return GMS_ERR_STATE;
    if (!s->dry_run) {
        Driver *d = driver();
        const CUmemAllocationProp prop = slab_prop(s->device, s->shareable);
        size_t done = 0;
        int rc = GMS_OK;
        for (; done < s->slabs.size() && rc == GMS_OK; ++done) {
            Slab &slab = s->slabs[done];
            const CUresult r = d->memCreate(&slab.handle, slab.size, &prop, 0);
            if (r != CUDA_SUCCESS) {
                rc = r == CUDA_ERROR_OUT_OF_MEMORY ? GMS_ERR_NOMEM : GMS_ERR_CUDA;
                break;
            }
            rc = map_slab(s, slab, true);
            if (rc != GMS_OK) {
                (void)d->memUnmap((CUdeviceptr)slab.va, slab.size);  // in case the mapping was made and only the access failed
                d->memRelease(slab.handle);
                slab.handle = 0;
                break;
            }
        }
        if (rc != GMS_OK) {  // undo: the service stays without pages, every address still reserved
            for (size_t i = 0; i < done; ++i) {
                d->memUnmap((CUdeviceptr)s->slabs[i].va, s->slabs[i].size);
                d->memRelease(s->slabs[i].handle);
                s->slabs[i].handle = 0;
            }
            return rc;
        }
    }
    s->backed = true;
    return GMS_OK;
}

int gms_service_acquire_ro(gms_service *s)
{
    if (!s) return GMS_ERR_NULL;
    std::lock_guard<std::mutex> l(s->mu);
    if ((s->state != GMS_STATE_COMMITTED && s->state != GMS_STATE_RO) || !s->attached) return GMS_ERR_STATE;
    s->state = GMS_STATE_RO;
    ++s->readers;
    return GMS_OK;
}

int gms_service_release_ro(gms_service *s)
{
    if (!s) return GMS_ERR_NULL;
    std::lock_guard<std::mutex> l(s->mu);
    if (s->state != GMS_STATE_RO || s->readers == 0) return GMS_ERR_STATE;
    if (--s->readers == 0) s->state = GMS_STATE_COMMITTED;
    return GMS_OK;
}

int gms_service_info(gms_service *s, gms_service_stats *out)
{
    if (!s || !out) return GMS_ERR_NULL;
    std::lock_guard<std::mutex> l(s->mu);
    gms_service_stats st = {};
    st.state = s->state;
    st.readers = s->readers;
    st.n_slabs = s->slabs.size();
    st.slab_bytes = s->slab_bytes;
    st.attached = s->attached ? 1u : 0u;
    st.backed = s->backed ? 1u : 0u;
    for (const Slab &slab : s->slabs) {
        st.bytes_reserved += slab.size;
        st.bytes_allocated += slab.used;
        if (slab.dedicated) ++st.n_dedicated;
    }
    *out = st;
    return GMS_OK;
}

int gms_service_access(gms_service *s, const void *dptr, uint32_t *writable)
{
    if (!s || !dptr || !writable) return GMS_ERR_NULL;
    std::lock_guard<std::mutex> l(s->mu);
    const uint64_t p = reinterpret_cast<uint64_t>(dptr);
    for (const Slab &slab : s->slabs) {
        if (p < slab.va || p >= slab.va + slab.size) continue;
        if (!s->attached || !s->backed) return GMS_ERR_STATE;  // the address is reserved but nothing is mapped there
        if (s->dry_run) {
            *writable = s->state == GMS_STATE_RW ? 1u : 0u;
            return GMS_OK;
        }
        CUmemLocation loc = {};
        loc.type = CU_MEM_LOCATION_TYPE_DEVICE;
        loc.id = s->device;
        unsigned long long flags = 0;
        if (driver()->memGetAccess(&flags, &loc, (CUdeviceptr)p) != CUDA_SUCCESS) return GMS_ERR_CUDA;
        *writable = flags == CU_MEM_ACCESS_FLAGS_PROT_READWRITE ? 1u : 0u;
        return GMS_OK;
    }
    return GMS_ERR_RANGE;  // not an address of this service
}

int gms_service_slab(gms_service *s, uint64_t index, gms_slab_info *out)
{
    if (!s || !out) return GMS_ERR_NULL;
    std::lock_guard<std::mutex> l(s->mu);
    if (index >= s->slabs.size()) return GMS_ERR_RANGE;
    const Slab &slab = s->slabs[index];
    gms_slab_info info = {};
    info.address = slab.va;
    info.bytes = slab.size;
    info.dedicated = slab.dedicated ? 1u : 0u;
    *out = info;
    return GMS_OK;
}

int gms_service_export_fd(gms_service *s, uint64_t index, int *fd)
{
    if (!s || !fd) return GMS_ERR_NULL;
    *fd = -1;
    std::lock_guard<std::mutex> l(s->mu);
    if (index >= s->slabs.size()) return GMS_ERR_RANGE;
    if (!s->shareable || s->dry_run || !s->backed) return GMS_ERR_STATE;
    int h = -1;
    if (driver()->memExportToShareableHandle(&h, s->slabs[index].handle, CU_MEM_HANDLE_TYPE_POSIX_FILE_DESCRIPTOR, 0) != CUDA_SUCCESS)
        return GMS_ERR_CUDA;
    *fd = h;
    return GMS_OK;
}

}  // extern "C"

// ---------------------------------------------------------------- the client's side
struct gms_import {
    struct Range {
        uint64_t va = 0, size = 0;
        CUmemGenericAllocationHandle handle = 0;
        bool mapped = false;
    };
    std::vector<Range> ranges;
};

extern "C" {

int gms_import_create(const int *fds, const gms_slab_info *slabs, size_t n, uint32_t flags, gms_import **out)
{
    if (!out || (n && (!fds || !slabs))) return GMS_ERR_NULL;
    *out = nullptr;
    if (flags & ~(GMS_IMPORT_WRITABLE | GMS_IMPORT_SAME_ADDRESS)) return GMS_ERR_ARG;
    cudaError_t e = cudaFree(nullptr);  // make sure the primary context exists and is current
    int device = 0;
    if (e == cudaSuccess) e = cudaGetDevice(&device);
    if (e != cudaSuccess) return gms::report_cuda_error(e);
    Driver *d = driver();
    if (!d->ok) return GMS_ERR_CUDA;
    gms_import *imp = new (std::nothrow) gms_import();
    if (!imp) return GMS_ERR_NOMEM;
    int rc = GMS_OK;
    try {
        imp->ranges.reserve(n);
    } catch (const std::bad_alloc &) {
        delete imp;
        return GMS_ERR_NOMEM;
    }
    for (size_t i = 0; i < n && rc == GMS_OK; ++i) {
        gms_import::Range r;
        r.size = slabs[i].bytes;
        if (fds[i] < 0 || r.size == 0) {
            rc = GMS_ERR_ARG;
            break;
        }
        if (d->memImportFromShareableHandle(&r.handle, reinterpret_cast<void *>(static_cast<uintptr_t>(fds[i])),
                                            CU_MEM_HANDLE_TYPE_POSIX_FILE_DESCRIPTOR) != CUDA_SUCCESS) {
            rc = GMS_ERR_CUDA;
            break;
        }
        // the service's address is asked for; whether any other one will do is the caller's choice
        CUdeviceptr va = 0;
        if (d->memAddressReserve(&va, r.size, 0, (CUdeviceptr)slabs[i].address, 0) != CUDA_SUCCESS) {
            d->memRelease(r.handle);
            rc = GMS_ERR_CUDA;
            break;
        }
        r.va = (uint64_t)va;
        imp->ranges.push_back(r);  // from here on gms_import_destroy undoes it
        if ((flags & GMS_IMPORT_SAME_ADDRESS) && r.va != slabs[i].address) {
            rc = GMS_ERR_RANGE;
            break;
        }
        if (d->memMap(va, r.size, 0, r.handle, 0) != CUDA_SUCCESS) {
            rc = GMS_ERR_CUDA;
            break;
        }
        imp->ranges.back().mapped = true;
        CUmemAccessDesc desc = {};
        desc.location.type = CU_MEM_LOCATION_TYPE_DEVICE;
        desc.location.id = device;
        desc.flags = (flags & GMS_IMPORT_WRITABLE) ? CU_MEM_ACCESS_FLAGS_PROT_READWRITE : CU_MEM_ACCESS_FLAGS_PROT_READ;
        if (d->memSetAccess(va, r.size, &desc, 1) != CUDA_SUCCESS) rc = GMS_ERR_CUDA;
    }
    if (rc != GMS_OK) {
        (void)gms_import_destroy(imp);
        return rc;
    }
    *out = imp;
    return GMS_OK;
}

int gms_import_address(const gms_import *imp, size_t index, void **dptr)
{
    if (!imp || !dptr) return GMS_ERR_NULL;
    if (index >= imp->ranges.size()) return GMS_ERR_RANGE;
    *dptr = reinterpret_cast<void *>(imp->ranges[index].va);
    return GMS_OK;
}

int gms_import_destroy(gms_import *imp)
{
    if (!imp) return GMS_OK;
    int rc = GMS_OK;
    if (!imp->ranges.empty()) {
        cudaError_t e = cudaDeviceSynchronize();  // nothing of this process may still be using the mappings
        if (e != cudaSuccess) rc = gms::report_cuda_error(e);
    }
    Driver *d = driver();
    for (gms_import::Range &r : imp->ranges) {
        if (r.mapped && d->memUnmap((CUdeviceptr)r.va, r.size) != CUDA_SUCCESS) rc = GMS_ERR_CUDA;
        if (r.va && d->memAddressFree((CUdeviceptr)r.va, r.size) != CUDA_SUCCESS) rc = GMS_ERR_CUDA;
        if (r.handle && d->memRelease(r.handle) != CUDA_SUCCESS) rc = GMS_ERR_CUDA;
    }
    delete imp;
    return rc;
}

}  // extern "C"
