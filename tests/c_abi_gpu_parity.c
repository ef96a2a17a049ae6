/*
 * Parity of the CUDA library against the CPU oracle from a plain C program: no Python, no torch.
 * Device memory comes from the CUDA runtime directly, the library is called through gms.h, the oracle
 * through its exported C functions (declared below as the oracle's source defines them).  Built and
 * run by tests/test_c_abi_client.py on a GPU machine.  Everything compared is integer data: bit-exact.
 */
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <cuda_runtime_api.h>

#include "gms.h"

typedef struct { uint64_t tensor_id, src_offset, dst_offset, nbytes; } gmso_entry;
typedef struct { uint64_t tensor_id, block; } gmso_mismatch;
int gmso_restore(const gmso_entry *e, size_t n, const uint8_t *image, uint64_t image_bytes, uint8_t *dst_base,
                 uint64_t dst_bytes, uint64_t *block_digests, uint64_t *tensor_digests);
int gmso_digest(const gmso_entry *e, size_t n, const uint8_t *dst_base, uint64_t dst_bytes, uint64_t *block_digests,
                uint64_t *tensor_digests);
uint64_t gmso_verify(const gmso_entry *e, size_t n, const uint64_t *computed, const uint64_t *expected,
                     gmso_mismatch *out, uint64_t cap);

#define CHECK(cond)                                                          \
    do {                                                                     \
        if (!(cond)) {                                                       \
            fprintf(stderr, "line %d: check failed: %s (cuda: %s)\n", __LINE__, #cond, gms_last_cuda_error()); \
            return 1;                                                        \
        }                                                                    \
    } while (0)

enum { N = 41, CAP = 8 };

static uint64_t rng_state = 0x2545F4914F6CDD1DULL; /* xorshift64: input generator only */
static uint64_t rnd(void)
{
    rng_state ^= rng_state << 13;
    rng_state ^= rng_state >> 7;
    rng_state ^= rng_state << 17;
    return rng_state;
}

int main(void)
{
    gmso_entry oe[N];
    gms_entry ge[N];
    uint64_t image_bytes = 0, slab_bytes = 0, n_blocks = 0, i;
    uint8_t *h_image, *h_slab, *h_want, *d_image, *d_slab;
    uint64_t *h_bd, *h_td, *w_bd, *w_td, *w_bd2, *w_td2, *d_bd, *d_td, *d_count, h_count = 0;
    gms_mismatch *d_out, h_out[CAP];
    gmso_mismatch w_out[CAP];
    gms_manifest *m = NULL;
    uint64_t nt, nb, payload, status = 99, w_count;

    /* layout: sizes from a few bytes to ~1.2 MB incl. 0, 4096 and odd tails; sources packed in order,
     * destinations laid out in reverse order with 256-byte guard gaps */
    for (i = 0; i < N; ++i) {
        uint64_t n = (i == 3) ? 0 : (i == 5) ? 4096 : (i % 7 == 0) ? 1200000 + rnd() % 4096 : 1 + rnd() % 70000;
        oe[i].tensor_id = 1000 + 3 * i;
        oe[i].src_offset = image_bytes;
        oe[i].nbytes = n;
        image_bytes += (n + 15) & ~(uint64_t)15;
        n_blocks += (n + 4095) / 4096;
    }
    for (i = N; i-- > 0;) {
        slab_bytes += 256;
        oe[i].dst_offset = slab_bytes;
        slab_bytes += (oe[i].nbytes + 15) & ~(uint64_t)15;
    }
    slab_bytes += 256;

    h_image = malloc(image_bytes); h_slab = malloc(slab_bytes); h_want = malloc(slab_bytes);
    h_bd = malloc(8 * n_blocks); w_bd = malloc(8 * n_blocks); w_bd2 = malloc(8 * n_blocks);
    h_td = malloc(8 * N); w_td = malloc(8 * N); w_td2 = malloc(8 * N);
    CHECK(h_image && h_slab && h_want && h_bd && w_bd && w_bd2 && h_td && w_td && w_td2);
    for (i = 0; i < image_bytes; ++i) h_image[i] = (uint8_t)(rnd() >> 56);

    CHECK(cudaMalloc((void **)&d_image, image_bytes) == cudaSuccess);
    CHECK(cudaMalloc((void **)&d_slab, slab_bytes) == cudaSuccess);
    CHECK(cudaMalloc((void **)&d_bd, 8 * n_blocks) == cudaSuccess && cudaMalloc((void **)&d_td, 8 * N) == cudaSuccess);
    CHECK(cudaMalloc((void **)&d_out, sizeof(gms_mismatch) * CAP) == cudaSuccess);
    CHECK(cudaMalloc((void **)&d_count, 8) == cudaSuccess);
    CHECK(cudaMemcpy(d_image, h_image, image_bytes, cudaMemcpyHostToDevice) == cudaSuccess);
    CHECK(cudaMemset(d_slab, 0xEE, slab_bytes) == cudaSuccess);
    memset(h_want, 0xEE, slab_bytes);

    for (i = 0; i < N; ++i) {
        ge[i].tensor_id = oe[i].tensor_id;
        ge[i].src_offset = oe[i].src_offset;
        ge[i].dst = d_slab + oe[i].dst_offset;
        ge[i].nbytes = oe[i].nbytes;
    }
    CHECK(gms_manifest_build(ge, N, image_bytes, 0, &m) == GMS_OK);
    CHECK(gms_manifest_info(m, &nt, &nb, &payload) == GMS_OK && nt == N && nb == n_blocks);

    /* restore: bytes (guard gaps included), block digests, tensor digests */
    CHECK(gms_restore(m, d_image, GMS_SRC_DEVICE, d_bd, d_td, NULL) == GMS_OK);
    CHECK(cudaDeviceSynchronize() == cudaSuccess);
    CHECK(gms_last_device_status(m, NULL, &status) == GMS_OK && status == 0);
    CHECK(cudaMemcpy(h_slab, d_slab, slab_bytes, cudaMemcpyDeviceToHost) == cudaSuccess);
    CHECK(cudaMemcpy(h_bd, d_bd, 8 * n_blocks, cudaMemcpyDeviceToHost) == cudaSuccess);
    CHECK(cudaMemcpy(h_td, d_td, 8 * N, cudaMemcpyDeviceToHost) == cudaSuccess);
    CHECK(gmso_restore(oe, N, h_image, image_bytes, h_want, slab_bytes, w_bd, w_td) == 0);
    CHECK(memcmp(h_slab, h_want, slab_bytes) == 0);
    CHECK(memcmp(h_bd, w_bd, 8 * n_blocks) == 0 && memcmp(h_td, w_td, 8 * N) == 0);

    /* commit the digests, damage two bytes from the host, digest in place, verify */
    CHECK(gms_manifest_set_expected(m, d_bd, NULL) == GMS_OK);
    {
        const uint64_t where[2] = {oe[7].dst_offset + 5000, oe[30].dst_offset};
        for (i = 0; i < 2; ++i) {
            h_want[where[i]] ^= 0x10;
            CHECK(cudaMemcpy(d_slab + where[i], h_want + where[i], 1, cudaMemcpyHostToDevice) == cudaSuccess);
        }
    }
    CHECK(gms_digest(m, d_bd, d_td, NULL) == GMS_OK);
    CHECK(gms_verify(m, d_bd, d_out, CAP, d_count, NULL) == GMS_OK);
    CHECK(cudaDeviceSynchronize() == cudaSuccess);
    CHECK(cudaMemcpy(h_bd, d_bd, 8 * n_blocks, cudaMemcpyDeviceToHost) == cudaSuccess);
    CHECK(cudaMemcpy(h_td, d_td, 8 * N, cudaMemcpyDeviceToHost) == cudaSuccess);
    CHECK(cudaMemcpy(&h_count, d_count, 8, cudaMemcpyDeviceToHost) == cudaSuccess);
    CHECK(cudaMemcpy(h_out, d_out, sizeof h_out, cudaMemcpyDeviceToHost) == cudaSuccess);
    CHECK(gmso_digest(oe, N, h_want, slab_bytes, w_bd2, w_td2) == 0);
    CHECK(memcmp(h_bd, w_bd2, 8 * n_blocks) == 0 && memcmp(h_td, w_td2, 8 * N) == 0);
    w_count = gmso_verify(oe, N, w_bd2, w_bd, w_out, CAP);
    CHECK(w_count == 2 && h_count == w_count);
    for (i = 0; i < w_count; ++i) CHECK(h_out[i].tensor_id == w_out[i].tensor_id && h_out[i].block == w_out[i].block);
    CHECK(h_out[0].tensor_id == oe[7].tensor_id && h_out[0].block == 1 && h_out[1].tensor_id == oe[30].tensor_id);

    /* the same decision in one pass: gms_digest_verify reports the digests and the list of the two calls above */
    CHECK(cudaMemset(d_bd, 0, 8 * n_blocks) == cudaSuccess && cudaMemset(d_out, 0, sizeof(gms_mismatch) * CAP) == cudaSuccess);
    CHECK(gms_digest_verify(m, d_bd, d_td, d_out, CAP, d_count, NULL) == GMS_OK);
    CHECK(cudaDeviceSynchronize() == cudaSuccess);
    CHECK(cudaMemcpy(h_bd, d_bd, 8 * n_blocks, cudaMemcpyDeviceToHost) == cudaSuccess);
    CHECK(cudaMemcpy(&h_count, d_count, 8, cudaMemcpyDeviceToHost) == cudaSuccess);
    CHECK(cudaMemcpy(h_out, d_out, sizeof h_out, cudaMemcpyDeviceToHost) == cudaSuccess);
    CHECK(memcmp(h_bd, w_bd2, 8 * n_blocks) == 0 && h_count == w_count);
    for (i = 0; i < w_count; ++i) CHECK(h_out[i].tensor_id == w_out[i].tensor_id && h_out[i].block == w_out[i].block);

    /* gms_restore_verify puts the image back over the damage: the oracle's restore digests again, nothing differs */
    CHECK(gms_restore_verify(m, d_image, GMS_SRC_DEVICE, d_bd, d_td, d_out, CAP, d_count, NULL) == GMS_OK);
    CHECK(cudaDeviceSynchronize() == cudaSuccess);
    CHECK(gms_last_device_status(m, NULL, &status) == GMS_OK && status == 0);
    CHECK(cudaMemcpy(h_slab, d_slab, slab_bytes, cudaMemcpyDeviceToHost) == cudaSuccess);
    CHECK(cudaMemcpy(h_bd, d_bd, 8 * n_blocks, cudaMemcpyDeviceToHost) == cudaSuccess);
    CHECK(cudaMemcpy(h_td, d_td, 8 * N, cudaMemcpyDeviceToHost) == cudaSuccess);
    CHECK(cudaMemcpy(&h_count, d_count, 8, cudaMemcpyDeviceToHost) == cudaSuccess);
    CHECK(gmso_restore(oe, N, h_image, image_bytes, h_want, slab_bytes, w_bd2, w_td2) == 0);
    CHECK(memcmp(h_slab, h_want, slab_bytes) == 0);
    CHECK(memcmp(h_bd, w_bd2, 8 * n_blocks) == 0 && memcmp(h_td, w_td2, 8 * N) == 0);
    CHECK(h_count == gmso_verify(oe, N, w_bd2, w_bd, w_out, CAP) && h_count == 0);

    CHECK(gms_manifest_destroy(m) == GMS_OK);
    cudaFree(d_image); cudaFree(d_slab); cudaFree(d_bd); cudaFree(d_td); cudaFree(d_out); cudaFree(d_count);
    printf("c abi gpu parity: ok (%d tensors, %llu blocks, %llu launches)\n", (int)N, (unsigned long long)n_blocks,
           (unsigned long long)gms_kernel_launches());
    return 0;
}
