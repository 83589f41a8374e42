// fosgd_decode_noalloc: the one-worker decoder for callers that cannot provide scratch memory.
//
// Some hosts of this library may not allocate device memory at the point where they decode:
// code running inside another framework's memory pool with no allocator hook exposed, a
// latency-critical loop that has banned cudaMalloc because it synchronises the device, or a
// process that has handed all remaining memory to something else.  For them the scratch
// buffer that fosgd_decode takes from the caller lives here instead, in a fixed device array
// that is part of the library image: every GPU that loads the library holds these
// FOSGD_NOALLOC_SCRATCH_BYTES until the process exits.
#include <mutex>

#include <cuda_runtime.h>

#include "../../include/fosgd.h"
#include "common.cuh"

namespace {

constexpr size_t kScratchBytes = FOSGD_NOALLOC_SCRATCH_BYTES;
constexpr int kMaxDevices = 64;

// The scratch itself.  In host code this name is only a handle for the runtime, not a device
// address: the address a kernel can use comes from cudaGetSymbolAddress, per device.
static __device__ __align__(256) unsigned char g_scratch[kScratchBytes];

std::mutex g_mutex;
void* g_scratch_ptr[kMaxDevices] = {};

// Device address of the scratch array on the current device, looked up once per device.
cudaError_t scratch_address(void** out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (g_scratch_ptr[dev] == nullptr) {
        void* ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_ptr[dev] = ptr;
    }
    *out = g_scratch_ptr[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" int fosgd_decode_noalloc(const uint32_t* bits, int64_t d, uint32_t worker_id, uint64_t seed,
                                    uint64_t step, float lambda, int block_log2, float* out,
                                    fosgd_stream stream)
{
    // the decoder's own argument checks come first, so that a bad pointer reads as such at any size
    int st = fosgd::check_decode_args(bits, d, lambda, block_log2, out);
    if (st != FOSGD_OK) return st;
    size_t need = 0;
    st = fosgd_workspace_bytes(FOSGD_OP_DECODE, d, 1, FOSGD_F32, block_log2, 1, &need);
    if (st != FOSGD_OK) return st;
    if (need > kScratchBytes) return FOSGD_ELIMIT;
    void* ptr = nullptr;
    if (need > 0) {
        const cudaError_t e = scratch_address(&ptr);
        if (e != cudaSuccess) {
            fosgd::set_last_cuda_error((int)e);
            return FOSGD_ECUDA;
        }
    }
    // The decoder overwrites every scratch entry it later reads, so nothing has to be cleared
    // between calls even though the array keeps what the previous call left in it.
    return fosgd_decode(bits, d, worker_id, seed, step, lambda, block_log2, out, ptr, need ? kScratchBytes : 0,
                        stream);
}
