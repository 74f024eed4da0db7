// kla_chunk_fwd_static_scratch: the chunk forward for callers that cannot allocate device memory.
//
// Some callers have no allocator to turn to when kla_chunk_fwd asks for a workspace: code running inside a
// region where the framework forbids or cannot serve allocations (an inference server with a fixed memory plan,
// a callback on a stream, a plugin handed only its input and output buffers), or a host program written in a
// language binding that exposes no cudaMalloc.  For them the scratch of the segment-parallel scan lives here, in
// a device array that is part of the library image: every GPU that loads the library sets KLA_STATIC_SCRATCH_BYTES
// aside until the process exits, and in exchange this entry point never allocates or frees anything.
#include <mutex>

#include "common.cuh"

namespace {

// The scratch itself.  In host code this name is only a handle for the runtime, not a device address: the
// address each device gave the array is looked up once with cudaGetSymbolAddress and that pointer is what the
// kernels receive.
static __device__ __align__(256) unsigned char g_static_scratch[KLA_STATIC_SCRATCH_BYTES];

constexpr int MAX_DEVICES = 64;
std::mutex g_mutex;
void *g_scratch_ptr[MAX_DEVICES] = {};

// Device address of the array on the current device; looked up on the first call per device.
kla_status scratch_for_current_device(void **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return KLA_ERR_DEVICE;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_scratch_ptr[dev]) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) {
            (void)cudaGetLastError();
            return KLA_ERR_DEVICE;
        }
        g_scratch_ptr[dev] = ptr;
    }
    *out = g_scratch_ptr[dev];
    return KLA_OK;
}

}  // namespace

extern "C" kla_status kla_chunk_fwd_static_scratch(const kla_desc *desc, const void *q, const void *k, const void *v,
                                                   const float *log_alpha, const float *eta, float eps, int32_t chunk,
                                                   const float *init_state, void *out, float *final_state)
{
    if (!desc) return KLA_ERR_NULL;
    kla_desc d = *desc;
    d.workspace = nullptr;
    d.workspace_bytes = 0;
    // the same argument checks as kla_chunk_fwd, in the same order, before anything about the scratch
    const kla_status vst = kla::check_chunk_args(&d, q, k, v, log_alpha, eta, eps, chunk, init_state, out, final_state, false);
    if (vst != KLA_OK) return vst;
    // what this shape needs (0 when sequences are not cut into segments); decided on the host, nothing launched
    const size_t need = kla_chunk_fwd_workspace_bytes(&d, chunk);
    if (need > (size_t)KLA_STATIC_SCRATCH_BYTES) return KLA_ERR_WORKSPACE;
    if (need > 0) {
        void *ptr = nullptr;
        const kla_status st = scratch_for_current_device(&ptr);
        if (st != KLA_OK) return st;
        d.workspace = ptr;
        d.workspace_bytes = KLA_STATIC_SCRATCH_BYTES;
    }
    // Every byte of the scratch that a call reads it has written first (segment bounds, per-segment maps and
    // states), so nothing has to be cleared between calls.
    return kla_chunk_fwd(&d, q, k, v, log_alpha, eta, eps, chunk, init_state, out, final_state);
}
