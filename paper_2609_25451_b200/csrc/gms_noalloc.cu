// gms_verify_flat_noalloc: the digest comparison of gms_verify for callers that
// must not allocate device memory.
//
// gms_verify keeps its per-segment counters and offsets (the scratch of the ordered
// compaction) and its block-base / tensor-id tables in memory that gms_manifest_build
// obtained with cudaMalloc.  Here the same tables live in one file-scope __device__
// array of fixed size, so the call needs no manifest and no allocation: the verify
// kernels are the same ones, handed pointers into that array.
//
// The array is a device symbol.  In host code its name is only a host-side stand-in,
// not a device address, so the host asks the runtime for the real address once per
// device (cudaGetSymbolAddress, with that device current) and passes that pointer to
// the kernels.  Device code in this file (the set-up kernel) names the array directly.
#include <mutex>

#include "../../include/gms.h"
#include "gms_internal.h"

namespace {

constexpr uint64_t kMaxBlocks = GMS_NOALLOC_MAX_BLOCKS;
constexpr uint32_t kMaxSegments = (uint32_t)(kMaxBlocks / gms::kVerifySegBlocks);
static_assert(kMaxBlocks % gms::kVerifySegBlocks == 0, "capacity must be a whole number of segments");

struct Scratch {
    uint64_t block_base[2];             // {0, n_blocks}: the one "tensor" of a flat comparison
    uint64_t tensor_id[2];              // [0] = the id to report; [1] unused
    uint32_t seg_count[kMaxSegments];   // differing slots per segment
};

// ~8 KiB per GPU that loads the library, held until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_scratch[sizeof(Scratch)];

// Rewrites the small tables for this call and clears the per-segment words the call will use
// (the array keeps whatever the previous call left in it).
__global__ void gms_noalloc_setup_kernel(uint64_t n_blocks, uint64_t tensor_id, uint32_t n_segments)
{
    Scratch *s = reinterpret_cast<Scratch *>(g_noalloc_scratch);
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i == 0) {
        s->block_base[0] = 0;
        s->block_base[1] = n_blocks;
        s->tensor_id[0] = tensor_id;
        s->tensor_id[1] = 0;
    }
    for (uint32_t k = i; k < n_segments; k += gridDim.x * blockDim.x) s->seg_count[k] = 0;
}

std::mutex g_mu;
constexpr int kMaxDevices = 64;
Scratch *g_dev_ptr[kMaxDevices];  // device address of g_noalloc_scratch, per device

}  // namespace

extern "C" int gms_verify_flat_noalloc(const uint64_t *d_computed, const uint64_t *d_expected, uint64_t n_blocks,
                                       uint64_t tensor_id, gms_mismatch *d_out, uint32_t cap, uint64_t *d_count, void *stream)
{
    if (!d_count || (cap && !d_out) || (n_blocks && (!d_computed || !d_expected))) return GMS_ERR_NULL;
    if (n_blocks > kMaxBlocks) return GMS_ERR_TOO_LARGE;
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return gms::report_cuda_error(e);
    if (dev < 0 || dev >= kMaxDevices) return GMS_ERR_ARG;
    Scratch *scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_mu);
        if (!g_dev_ptr[dev]) {  // first call on this device: resolve the symbol's device address
            void *p = nullptr;
            e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
            if (e != cudaSuccess) return gms::report_cuda_error(e);
            g_dev_ptr[dev] = static_cast<Scratch *>(p);
        }
        scratch = g_dev_ptr[dev];
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const uint32_t n_segments = (uint32_t)((n_blocks + gms::kVerifySegBlocks - 1) / gms::kVerifySegBlocks);
    gms_noalloc_setup_kernel<<<n_segments > 256 ? 8 : 1, 256, 0, s>>>(n_blocks, tensor_id, n_segments);
    if ((e = cudaGetLastError()) != cudaSuccess) return gms::report_cuda_error(e);
    gms::count_launches(1);

    gms::VerifyArgs a = {};
    a.computed = d_computed;
    a.expected = d_expected;
    a.n_blocks = n_blocks;
    a.block_base = scratch->block_base;  // address arithmetic on the device pointer only; nothing is dereferenced here
    a.tensor_ids = scratch->tensor_id;
    a.n_tensors = 1;
    a.seg_count = scratch->seg_count;
    a.n_segments = n_segments;
    a.out = d_out;
    a.cap = cap;
    a.count = d_count;
    if ((e = gms::launch_verify(a, s)) != cudaSuccess) return gms::report_cuda_error(e);
    return GMS_OK;
}
