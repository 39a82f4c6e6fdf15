// lamp_conv3d_dgrad_static_scratch: the data-gradient pass for callers that cannot hand the library
// a workspace because they cannot allocate device memory at the point of the call - for example a
// layer plugged into an inference or training engine that gave out all device memory at start-up, or
// a latency-critical loop in which cudaMalloc (which synchronises the device and may fail under
// memory pressure) is not allowed.  The scratch the pass needs - the transposed copy of the weights -
// lives in a fixed array inside the library image instead.
#include "common.cuh"

namespace {

// Scratch for the transposed weights, 27 * c_in * c_out bf16 values.  Every GPU that loads the library
// holds these bytes until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[LAMP_STATIC_SCRATCH_BYTES];

constexpr int MAX_DEVICES = 64;
// device address of g_static_scratch, per device, resolved on first use.  Host threads may race to fill an entry:
// all of them store the same value, and the accesses are atomic.  The cached address belongs to the device's
// primary context: it does not survive a cudaDeviceReset of that device.
void *g_scratch_addr[MAX_DEVICES];

// In host code `g_static_scratch` is only a handle of the symbol, not an address a kernel may use:
// the device address has to be asked for, with the device in question current.
lamp_status_t scratch_for_current_device(void **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return LAMP_ERR_CUDA;
    void *p = __atomic_load_n(&g_scratch_addr[dev], __ATOMIC_ACQUIRE);
    if (!p) {
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return LAMP_ERR_CUDA;
        __atomic_store_n(&g_scratch_addr[dev], p, __ATOMIC_RELEASE);
    }
    *out = p;
    return LAMP_OK;
}

}  // namespace

extern "C" lamp_status_t lamp_conv3d_dgrad_static_scratch(const lamp_conv_desc_t *desc, const lamp_tensor_t *dy,
                                                          const void *w, lamp_tensor_t *dx, void *cuda_stream)
{
    if (!desc || !dy || !w || !dx) return LAMP_ERR_INVALID_ARG;
    const size_t need = lamp_conv3d_workspace_min_bytes(desc, dx, LAMP_PASS_DGRAD);
    if (need > (size_t)LAMP_STATIC_SCRATCH_BYTES) return LAMP_ERR_SCRATCH_LIMIT;
    void *scratch = nullptr;
    const lamp_status_t s = scratch_for_current_device(&scratch);
    if (s != LAMP_OK) return s;
    // Nothing in the scratch has to start at zero: the pass overwrites the part it reads.
    // Exactly the smallest workspace is handed on, so the pass runs as lamp_conv3d_dgrad does with that workspace
    // (reduction not split) whatever the layer's size: same kernels, same bits.
    return lamp_conv3d_dgrad(desc, dy, w, dx, scratch, need, cuda_stream);
}
