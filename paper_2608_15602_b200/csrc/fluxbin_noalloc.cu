// fluxbin_linear_noalloc: the one-layer entry point for callers that own no scratch memory.
//
// The split-K accumulators and arrival counters that fluxbin_linear keeps in a caller-provided
// workspace live here in a fixed array inside the library image instead, so the caller passes
// nothing but the packed layer, the activations and the output.
#include "fluxbin_internal.h"

#include <cuda_runtime.h>
#include <mutex>

// Scratch shared by every call on a device; each GPU that loads the library holds it until exit.  A call
// needs fluxbin_workspace_size(w, B) bytes of it: 4 bytes per output row (padded to 32) and per accumulator
// row -- 1 at batch 1, 2 at batch 2, 4 from batch 3 (fp32 table entries) or 3..4 (fp16 entries), 8 from batch 5
// with fp16 entries -- plus a few hundred bytes of counters.  1 MiB therefore takes about 260,000 output rows
// at batch 1, 130,000 at batch 2, 65,000 with four accumulator rows and 32,000 with eight.
#define FLUXBIN_NOALLOC_SCRATCH_BYTES (1u << 20)
static __device__ __align__(256) unsigned char g_fluxbin_noalloc_scratch[FLUXBIN_NOALLOC_SCRATCH_BYTES];

namespace {

// Device address of the array above, per device.  The array's name is only a host-side handle for
// the symbol: the address a kernel can use has to be asked for, on the device that will run it.
void *g_scratch_ptr[fb::kMaxDevices];
bool g_scratch_ready[fb::kMaxDevices];
std::mutex g_scratch_mutex;

} // namespace

extern "C" size_t fluxbin_noalloc_capacity(void) { return FLUXBIN_NOALLOC_SCRATCH_BYTES; }

extern "C" fluxbin_status_t fluxbin_linear_noalloc(const fluxbin_weight_t *w, const uint16_t *d_x, int32_t B, int64_t ldx,
                                                   void *d_y, int32_t y_is_fp32, int64_t ldy, void *cuda_stream)
{
    // every argument check of fluxbin_linear that needs no device comes first: a rejected call puts nothing on the stream
    if (!w || !d_x || !d_y) return FLUXBIN_ERR_NULL;
    if (B < 1 || ldx < w->h.N || ldy < w->h.M) return FLUXBIN_ERR_RANGE;
    if ((((uintptr_t)d_x) & 15) || (((uintptr_t)d_y) & 15)) return FLUXBIN_ERR_ALIGNMENT;
    if (w->h.npairs[1] > 0 && w->h.sps[1] == 16 && w->h.sps[0] != 16) return FLUXBIN_ERR_FORMAT;
    const size_t need = fluxbin_workspace_size(w, B);
    if (need == 0) return FLUXBIN_ERR_RANGE;
    if (need > FLUXBIN_NOALLOC_SCRATCH_BYTES) return FLUXBIN_ERR_BUFFER_TOO_SMALL;   // layer too tall for the fixed scratch

    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fb::record_cuda_error((int)e);
    if (dev < 0 || dev >= fb::kMaxDevices) return FLUXBIN_ERR_UNSUPPORTED;
    if (dev != w->device) return FLUXBIN_ERR_UNSUPPORTED;      // the layer lives on another device than the current one
    void *scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_scratch_mutex);
        if (!g_scratch_ready[dev]) {
            void *p = nullptr;
            e = cudaGetSymbolAddress(&p, g_fluxbin_noalloc_scratch);
            if (e != cudaSuccess || !p) return fb::record_cuda_error((int)(e != cudaSuccess ? e : cudaErrorInvalidSymbol));
            g_scratch_ptr[dev] = p;
            g_scratch_ready[dev] = true;
        }
        scratch = g_scratch_ptr[dev];
    }
    // The array keeps whatever the last call left behind.  A call that ran to completion leaves it
    // zeroed, but one that was cut short does not, so the part this call uses is cleared first.
    e = cudaMemsetAsync(scratch, 0, need, (cudaStream_t)cuda_stream);
    if (e != cudaSuccess) return fb::record_cuda_error((int)e);
    return fluxbin_linear(w, d_x, B, ldx, d_y, y_is_fp32, ldy, scratch, need, cuda_stream);
}
