// Declarations shared by the host packer and the CUDA side of the library (not installed).
#ifndef FLUXBIN_INTERNAL_H
#define FLUXBIN_INTERNAL_H

#include "../../include/fluxbin.h"
#include "fluxbin_layout.h"

#include <atomic>
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
// dimension rules and the salient map (host pointer d->sal_idx) without looking at the other arrays
fluxbin_status_t validate_dims_and_map(const fluxbin_layer_desc_t *d);
// header, salient sub-vector list and the row-scale groups without salient columns of a validated description
void make_packed_header(const fluxbin_layer_desc_t *d, FbHeader &h, std::vector<SalSvec> &sv, std::vector<int> &dead);
// shared-memory opt-in of every instantiation of the layer kernel on the current device
fluxbin_status_t opt_in_all_kernels();
// remember a CUDA error code for fluxbin_last_cuda_error(), clear the runtime's sticky state, return FLUXBIN_ERR_CUDA
fluxbin_status_t record_cuda_error(int cuda_error);

constexpr int kMaxDevices = 64;
constexpr int kMaxGrid = 1024;             // CTAs per launch (a B200 runs 444 at most)
constexpr int kMaxSingleShares = 512;      // CTAs of a one-layer launch: its share bounds travel in the kernel parameters

// Launch shape and share bounds of a one-layer launch in one launch mode (see cut_launch in fluxbin_api.cu).
struct SingleLaunch {
    int grid, np;
    int cut[kMaxSingleShares + 1];
};

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
    int table_format;   // FLUXBIN_TABLES_FP32 / _FP16 / _FP32_MU4: how launches hold their table entries
    mutable std::atomic<fb::SingleLaunch *> single[9];   // per launch mode, made on first use, owned by the handle
};

#endif
