/*
 * A plain C99 client of the library's C ABI, built and run by tests/test_c_abi_client.py without a GPU.
 * It proves three things the Python binding cannot: the header is valid C (not only C++), every
 * function the header declares links against libgms.so with C linkage, and the host-only calls
 * (manifest validation and chunking, the service's dry-run backend, the error texts) work from C.
 * No call here touches a device.
 */
#include <stdio.h>
#include <string.h>

#include "gms.h"

#define CHECK(cond)                                                         \
    do {                                                                    \
        if (!(cond)) {                                                      \
            fprintf(stderr, "line %d: check failed: %s\n", __LINE__, #cond); \
            return 1;                                                       \
        }                                                                   \
    } while (0)

typedef void (*fn)(void);

int main(void)
{
    /* every declared entry point, taken by address: an undeclared or unexported name fails to link */
    const fn all[] = {
        (fn)gms_manifest_build, (fn)gms_manifest_destroy, (fn)gms_manifest_info, (fn)gms_manifest_block_base,
        (fn)gms_manifest_chunk_count, (fn)gms_manifest_chunk, (fn)gms_manifest_set_expected, (fn)gms_restore,
        (fn)gms_capture, (fn)gms_digest, (fn)gms_verify, (fn)gms_digest_verify, (fn)gms_restore_verify, (fn)gms_verify_tensors, (fn)gms_verify_flat_noalloc,
        (fn)gms_last_device_status, (fn)gms_kv_restore, (fn)gms_kv_capture, (fn)gms_kv_digest, (fn)gms_kv_verify, (fn)gms_host_image_alloc,
        (fn)gms_host_image_free, (fn)gms_pipe_create, (fn)gms_pipe_direct_io, (fn)gms_pipe_mapped_writes, (fn)gms_pipe_destroy, (fn)gms_restore_fd, (fn)gms_capture_fd, (fn)gms_stage_create,
        (fn)gms_stage_destroy, (fn)gms_restore_staged, (fn)gms_service_create, (fn)gms_service_destroy,
        (fn)gms_service_acquire_rw, (fn)gms_service_alloc, (fn)gms_service_commit, (fn)gms_service_abort,
        (fn)gms_service_acquire_ro, (fn)gms_service_release_ro, (fn)gms_service_info, (fn)gms_service_access,
        (fn)gms_service_detach, (fn)gms_service_reattach, (fn)gms_service_release_pages, (fn)gms_service_back_pages,
        (fn)gms_service_slab, (fn)gms_service_export_fd, (fn)gms_import_create, (fn)gms_import_address, (fn)gms_import_destroy,
        (fn)gms_launch_geometry, (fn)gms_kernel_launches, (fn)gms_set_device, (fn)gms_strerror, (fn)gms_last_cuda_error,
        (fn)gms_version,
    };
    size_t i;
    for (i = 0; i < sizeof all / sizeof all[0]; ++i) CHECK(all[i] != NULL);

    CHECK(sizeof(gms_entry) == 32 && sizeof(gms_mismatch) == 16);
    CHECK(gms_version() != 0);
    CHECK(strlen(gms_strerror(GMS_OK)) > 0 && strlen(gms_strerror(GMS_ERR_OVERLAP)) > 0);
    CHECK(strcmp(gms_strerror(GMS_ERR_ALIGN), gms_strerror(GMS_ERR_RANGE)) != 0);

    /* three tensors: 10000 bytes (3 blocks), 0 bytes (0 blocks), 4096 bytes (1 block) */
    {
        gms_entry e[3];
        gms_manifest *m = NULL;
        uint64_t nt = 0, nb = 0, payload = 0, base = 99, nc = 0, covered = 0, k;
        memset(e, 0, sizeof e);
        e[0].tensor_id = 7;  e[0].src_offset = 0;     e[0].dst = (void *)(uintptr_t)0x10000; e[0].nbytes = 10000;
        e[1].tensor_id = 8;  e[1].src_offset = 10000; e[1].dst = (void *)(uintptr_t)0x20000; e[1].nbytes = 0;
        e[2].tensor_id = 9;  e[2].src_offset = 10000; e[2].dst = (void *)(uintptr_t)0x30000; e[2].nbytes = 4096;
        CHECK(gms_manifest_build(e, 3, 14096, GMS_BUILD_HOST_ONLY, &m) == GMS_OK && m != NULL);
        CHECK(gms_manifest_info(m, &nt, &nb, &payload) == GMS_OK);
        CHECK(nt == 3 && nb == 4 && payload == 14096);
        CHECK(gms_manifest_block_base(m, 0, &base) == GMS_OK && base == 0);
        CHECK(gms_manifest_block_base(m, 1, &base) == GMS_OK && base == 3);
        CHECK(gms_manifest_block_base(m, 2, &base) == GMS_OK && base == 3);
        CHECK(gms_manifest_block_base(m, 3, &base) != GMS_OK);
        CHECK(gms_manifest_chunk_count(m, &nc) == GMS_OK && nc >= 2);
        for (k = 0; k < nc; ++k) {
            uint64_t entry = 99, off = 1, n = 0;
            CHECK(gms_manifest_chunk(m, k, &entry, &off, &n) == GMS_OK);
            CHECK(entry < 3 && n > 0 && off % GMS_BLOCK_BYTES == 0 && off + n <= e[entry].nbytes);
            covered += n;
        }
        CHECK(covered == payload);
        /* a host-only manifest refuses device work before anything is enqueued */
        CHECK(gms_digest(m, NULL, NULL, NULL) == GMS_ERR_STATE);
        CHECK(gms_manifest_destroy(m) == GMS_OK);

        /* validation: each defect has its own code, and *out stays NULL */
        m = NULL;
        e[2].src_offset = 10008;
        CHECK(gms_manifest_build(e, 3, 1 << 20, GMS_BUILD_HOST_ONLY, &m) == GMS_ERR_ALIGN && m == NULL);
        e[2].src_offset = 10000;
        CHECK(gms_manifest_build(e, 3, 14095, GMS_BUILD_HOST_ONLY, &m) == GMS_ERR_RANGE && m == NULL);
        e[2].dst = (void *)(uintptr_t)0x10010;
        CHECK(gms_manifest_build(e, 3, 14096, GMS_BUILD_HOST_ONLY, &m) == GMS_ERR_OVERLAP && m == NULL);
        e[2].dst = (void *)(uintptr_t)0x30000;
        e[2].tensor_id = 7;
        CHECK(gms_manifest_build(e, 3, 14096, GMS_BUILD_HOST_ONLY, &m) == GMS_ERR_DUP_ID && m == NULL);
        CHECK(gms_manifest_build(NULL, 3, 14096, GMS_BUILD_HOST_ONLY, &m) == GMS_ERR_NULL);
        CHECK(gms_manifest_build(NULL, 0, 0, GMS_BUILD_HOST_ONLY, &m) == GMS_OK && m != NULL); /* empty is legal */
        CHECK(gms_manifest_info(m, &nt, &nb, &payload) == GMS_OK && nt == 0 && nb == 0 && payload == 0);
        CHECK(gms_manifest_destroy(m) == GMS_OK);
    }

    /* the ownership state machine, on the dry-run backend (addresses only, no device) */
    {
        gms_service *s = NULL;
        gms_service_stats st;
        void *a = NULL, *b = NULL;
        uint32_t writable = 7;
        CHECK(gms_service_create(0, GMS_SERVICE_DRY_RUN, &s) == GMS_OK && s != NULL);
        CHECK(gms_service_alloc(s, 4096, &a) == GMS_ERR_STATE);   /* EMPTY: no writer yet */
        CHECK(gms_service_acquire_ro(s) == GMS_ERR_STATE);       /* nothing committed to read */
        CHECK(gms_service_acquire_rw(s) == GMS_OK);
        CHECK(gms_service_acquire_rw(s) == GMS_ERR_STATE);       /* one writer at a time */
        CHECK(gms_service_alloc(s, 1000, &a) == GMS_OK && a != NULL);
        CHECK(gms_service_alloc(s, 5000, &b) == GMS_OK && b != NULL && a != b);
        CHECK(((uintptr_t)a & 15u) == 0 && ((uintptr_t)b & 15u) == 0);
        CHECK(gms_service_access(s, a, &writable) == GMS_OK && writable == 1);
        CHECK(gms_service_commit(s) == GMS_OK);
        CHECK(gms_service_alloc(s, 16, &a) == GMS_ERR_STATE);     /* committed state is immutable */
        CHECK(gms_service_access(s, b, &writable) == GMS_OK && writable == 0);
        CHECK(gms_service_acquire_ro(s) == GMS_OK && gms_service_acquire_ro(s) == GMS_OK);
        CHECK(gms_service_acquire_rw(s) == GMS_ERR_STATE);       /* readers attached */
        CHECK(gms_service_info(s, &st) == GMS_OK);
        CHECK(gms_service_release_ro(s) == GMS_OK && gms_service_release_ro(s) == GMS_OK);
        CHECK(gms_service_release_ro(s) == GMS_ERR_STATE);
        CHECK(gms_service_destroy(s) == GMS_OK);
    }
    puts("c abi client: ok");
    return 0;
}
