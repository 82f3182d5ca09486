// dig_gla_fwd_static: the forward GLA call for callers that cannot allocate device memory.
//
// dig_gla_fwd keeps the segment states and decay factors in a workspace the caller allocates.
// Some callers have no allocator to ask: code that runs where cudaMalloc is forbidden or would
// stall (a real-time loop, a plugin whose host owns all device memory, a process working under a
// fixed memory budget).  For them the same scratch lives in a fixed-size array in device global
// memory that is part of this library's image.  A GPU holds those kScratchBytes from the moment the
// runtime loads this translation unit's module on it until the process exits: with lazy module
// loading that is the first call below on the device (the symbol look-up triggers it), with eager
// loading it is context creation.
#include <mutex>

#include "dig_common.cuh"

namespace {

constexpr size_t kScratchBytes = DIG_GLA_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

// In host code `g_static_scratch` is only a handle for the runtime's symbol table, not a device
// address, so the address is looked up once per device (with that device current) and cached.
constexpr int kMaxDevices = 64;
std::mutex g_mutex;
void *g_scratch_of_device[kMaxDevices] = {};

dig_status scratch_for_current_device(void **ptr)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return DIG_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (g_scratch_of_device[dev] == nullptr) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return DIG_ERR_CUDA;
        g_scratch_of_device[dev] = p;
    }
    *ptr = g_scratch_of_device[dev];
    return DIG_OK;
}

}  // namespace

extern "C" dig_status dig_gla_fwd_static(const void *q, const void *k, const void *v, const float *gate,
                                         void *out, int B, int H, int grid_h, int grid_w, int d_k,
                                         int d_v, int chunk, int direction, int dtype, void *cuda_stream)
{
    const size_t need = dig_gla_workspace_bytes(B, H, grid_h, grid_w, d_k, d_v, chunk, dtype, 0);
    if (need == 0) return DIG_ERR_INVALID_ARG;
    if (need > kScratchBytes) return DIG_ERR_SCRATCH_LIMIT;
    void *scratch = nullptr;
    const dig_status st = scratch_for_current_device(&scratch);
    if (st != DIG_OK) return st;
    // The forward kernels write every state and decay factor before reading it, so nothing in the
    // array has to be cleared between calls.
    return dig_gla_fwd(q, k, v, gate, out, B, H, grid_h, grid_w, d_k, d_v, chunk, direction, dtype,
                       scratch, kScratchBytes, cuda_stream);
}
