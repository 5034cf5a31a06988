// fluxbin_linear_noalloc: the one-layer entry point for callers that own no scratch memory.
//
// The split-K accumulators and arrival counters that fluxbin_linear keeps in a caller-provided
// workspace live here in a fixed array inside the library image instead, so the caller passes
// nothing but the packed layer, the activations and the output.
#include "fluxbin_internal.h"

#include <cuda_runtime.h>
#include <mutex>

// Scratch shared by every call on a device.  1 MiB covers any layer with up to 130,000 output rows at
// any batch size (260,000 rows at batch 1); each GPU that loads the library holds it until exit.
#define FLUXBIN_NOALLOC_SCRATCH_BYTES (1u << 20)
static __device__ __align__(256) unsigned char g_fluxbin_noalloc_scratch[FLUXBIN_NOALLOC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;
// Device address of the array above, per device.  The array's name is only a host-side handle for
// the symbol: the address a kernel can use has to be asked for, on the device that will run it.
void *g_scratch_ptr[kMaxDevices];
bool g_scratch_ready[kMaxDevices];
std::mutex g_scratch_mutex;

} // namespace

extern "C" size_t fluxbin_noalloc_capacity(void) { return FLUXBIN_NOALLOC_SCRATCH_BYTES; }

extern "C" fluxbin_status_t fluxbin_linear_noalloc(const fluxbin_weight_t *w, const uint16_t *d_x, int32_t B, int64_t ldx,
                                                   void *d_y, int32_t y_is_fp32, int64_t ldy, void *cuda_stream)
{
    if (!w || !d_x || !d_y) return FLUXBIN_ERR_NULL;
    if (B < 1) return FLUXBIN_ERR_RANGE;
    const size_t need = fluxbin_workspace_size(w, B);
    if (need == 0) return FLUXBIN_ERR_RANGE;
    if (need > FLUXBIN_NOALLOC_SCRATCH_BYTES) return FLUXBIN_ERR_BUFFER_TOO_SMALL;   // layer too tall for the fixed scratch

    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return FLUXBIN_ERR_CUDA;
    if (dev != w->device) return FLUXBIN_ERR_UNSUPPORTED;      // the layer lives on another device than the current one
    void *scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_scratch_mutex);
        if (!g_scratch_ready[dev]) {
            void *p = nullptr;
            if (cudaGetSymbolAddress(&p, g_fluxbin_noalloc_scratch) != cudaSuccess || !p) {
                (void)cudaGetLastError();
                return FLUXBIN_ERR_CUDA;
            }
            g_scratch_ptr[dev] = p;
            g_scratch_ready[dev] = true;
        }
        scratch = g_scratch_ptr[dev];
    }
    // The array keeps whatever the last call left behind.  A call that ran to completion leaves it
    // zeroed, but one that was cut short does not, so the part this call uses is cleared first.
    if (cudaMemsetAsync(scratch, 0, need, (cudaStream_t)cuda_stream) != cudaSuccess) {
        (void)cudaGetLastError();
        return FLUXBIN_ERR_CUDA;
    }
    return fluxbin_linear(w, d_x, B, ldx, d_y, y_is_fp32, ldy, scratch, need, cuda_stream);
}
