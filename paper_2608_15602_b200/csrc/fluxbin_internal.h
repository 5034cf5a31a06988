// Declarations shared by the host packer and the CUDA side of the library (not installed).
#ifndef FLUXBIN_INTERNAL_H
#define FLUXBIN_INTERNAL_H

#include "../../include/fluxbin.h"
#include "fluxbin_layout.h"

#include <vector>

namespace fb {

struct SalSvec {
    int vstart; // first virtual column
    int w;      // live columns (1..8); the rest of the sub-vector is zero padding
    int G;      // row-scale group of its columns
};

fluxbin_status_t validate_dims(const fluxbin_layer_desc_t *d);
void salient_svecs(const fluxbin_layer_desc_t *d, int sps1, std::vector<SalSvec> &out);
fluxbin_status_t check_header(const void *p, size_t bytes, FbHeader &h);
// remember a CUDA error code for fluxbin_last_cuda_error(), clear the runtime's sticky state, return FLUXBIN_ERR_CUDA
fluxbin_status_t record_cuda_error(int cuda_error);

} // namespace fb

// The opaque handle: a copy of the header plus the borrowed device pointer.
struct fluxbin_weight {
    FbHeader h;
    void *d_packed;
    size_t d_bytes;
    int device;
    int num_sms;
    int tile_rb;  // row blocks (of 32 rows) per arrival-counter tile
    int ntiles;
    int table_format;   // FLUXBIN_TABLES_FP32 / _FP16: how batched launches (B >= 2) hold their table entries
};

#endif
