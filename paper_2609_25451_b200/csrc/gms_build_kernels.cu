// Work-list expansion on the device.  gms_manifest_build validates the layout record on the host and computes, per
// tensor, where its chunks go in the list; the 32-byte chunk records themselves (a million for a 16 GB manifest)
// are written here, so that building a manifest costs the host work proportional to the number of tensors, not of
// chunks.  The order is that of a stable sort by length, longest first: all full-length chunks in entry order, then
// each tensor's short last chunk at the position the host ranked it at.
#include "gms_internal.h"

namespace gms {
namespace {

__global__ void gms_expand_chunks_kernel(ExpandArgs a)
{
    const uint64_t chunk_bytes = (uint64_t)a.chunk_blocks * kBlockBytes;
    const uint64_t total = a.n_full + a.n_tensors, step = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += step) {
        uint32_t t;  // slot of the tensor in the list's tensor order
        uint64_t off, pos;
        if (i < a.n_full) {
            // tensor t with full_base[t] <= i < full_base[t + 1] (tensors without a full chunk share a base)
            uint32_t lo = 0, hi = a.n_tensors;
            while (hi - lo > 1) {
                const uint32_t mid = lo + (hi - lo) / 2;
                if (a.full_base[mid] <= i) lo = mid; else hi = mid;
            }
            t = lo;
            off = (i - a.full_base[t]) * chunk_bytes;
            pos = i;
        } else {
            t = (uint32_t)(i - a.n_full);
            if (a.tail_pos[t] == 0xffffffffu) continue;  // the tensor ends on a chunk boundary (or is empty)
            off = (a.full_base[t + 1] - a.full_base[t]) * chunk_bytes;
            pos = a.tail_pos[t];
        }
        const uint32_t e = a.perm ? a.perm[t] : t;  // the entry
        const uint64_t nbytes = a.nbytes[e];
        Chunk c;
        c.src_off = a.src_offset[e] + off;
        c.dst = a.dst[e] + off;
        c.nbytes = (uint32_t)(nbytes - off < chunk_bytes ? nbytes - off : chunk_bytes);
        c.tensor = e;
        c.gblock0 = (uint32_t)(a.block_base[e] + off / kBlockBytes);
        c.tblock0 = (uint32_t)(off / kBlockBytes);
        a.out[pos] = c;
    }
}

}  // namespace

cudaError_t launch_expand_chunks(const ExpandArgs &a, cudaStream_t s)
{
    const uint64_t total = a.n_full + a.n_tensors;
    if (total == 0) return cudaSuccess;
    uint64_t blocks = (total + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    gms_expand_chunks_kernel<<<(uint32_t)blocks, 256, 0, s>>>(a);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace gms
