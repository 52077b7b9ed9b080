// mor_analyze_quantize_static: mor_analyze_quantize with the device scratch taken from an array
// that is part of the library image instead of a buffer the caller allocates.
//
// Who this is for: code that must not (or cannot) call cudaMalloc where it runs -- a callback
// inside somebody else's runtime that owns all device memory, a real-time loop in which an
// allocation's implicit device synchronisation is not acceptable, a process whose memory
// budget was fixed at start-up.  Such a caller still owns its inputs and outputs; only the
// scratch (an amax slot and a status word, then per 32 KiB tile of input one 40-byte partial result and
// the block keys that the amax pre-pass hands to the main kernel) comes from here.
#include <mutex>

#include "mor_internal.h"

namespace {

// Every GPU that loads the library holds this array until the process exits.
__device__ __align__(256) unsigned char g_static_scratch[MOR_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
void* g_scratch_ptr[kMaxDevices];     // device address of the array, per device; nullptr = not looked up yet
std::mutex g_scratch_mutex;

// In host code `g_static_scratch` names a host-side stand-in, not device memory, so the address a
// kernel can use has to be asked for, once per device, with that device current.
mor_status_t scratch_for_current_device(void** out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MOR_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (g_scratch_ptr[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return MOR_ERR_CUDA;
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return MOR_OK;
}

}  // namespace

extern "C" mor_status_t mor_analyze_quantize_static(const mor_tensor_desc_t* host_desc, const mor_outputs_t* host_out,
                                                    void* cuda_stream)
{
    if (host_desc == nullptr || host_out == nullptr) return MOR_ERR_INVALID_ARG;
    const size_t need = mor_workspace_bytes(host_desc, 1);
    if (need == 0) return MOR_ERR_UNSUPPORTED;                       // a block shape without a kernel
    if (need > (size_t)MOR_STATIC_SCRATCH_BYTES) return MOR_ERR_STATIC_SCRATCH;
    void* scratch = nullptr;
    const mor_status_t st = scratch_for_current_device(&scratch);
    if (st != MOR_OK) return st;
    return mor_analyze_quantize(host_desc, host_out, scratch, (size_t)MOR_STATIC_SCRATCH_BYTES, cuda_stream);
}
