// C-ABI entry points that touch the GPU: pack-to-device, attach, unpack-from-device, workspace,
// fluxbin_linear (launch only: no allocation, no synchronisation) and the table test hook.
#include "fluxbin_internal.h"
#include "fluxbin_kernel.cuh"

#include <cstdlib>
#include <cstring>
#include <atomic>
#include <mutex>
#include <vector>
#include <new>

using namespace fb;

static_assert(fb::kMaxSingleShares == fbk::kMaxSingleShares, "one-layer launches: host and kernel agree on the parameter array");

static thread_local int g_last_cuda_error = 0;

static fluxbin_status_t cuda_fail(cudaError_t e)
{
    g_last_cuda_error = (int)e;
    (void)cudaGetLastError();
    return FLUXBIN_ERR_CUDA;
}
#define FB_CUDA(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) return cuda_fail(e_); } while (0)

extern "C" int fluxbin_last_cuda_error(void) { return g_last_cuda_error; }

// the same bookkeeping for the library's other translation units
fluxbin_status_t fb::record_cuda_error(int cuda_error) { return cuda_fail((cudaError_t)cuda_error); }

extern "C" const char *fluxbin_status_string(fluxbin_status_t s)
{
    switch (s) {
    case FLUXBIN_OK: return "ok";
    case FLUXBIN_ERR_NULL: return "null pointer";
    case FLUXBIN_ERR_SHAPE: return "unsupported shape (need N%32==0, g%32==0, N%g==0, N<=65536, M>=1)";
    case FLUXBIN_ERR_RANGE: return "argument out of range";
    case FLUXBIN_ERR_SALIENT_MAP: return "salient map not strictly ascending in [0,N)";
    case FLUXBIN_ERR_BUFFER_TOO_SMALL: return "buffer too small";
    case FLUXBIN_ERR_ALIGNMENT: return "device pointer not 16-byte aligned";
    case FLUXBIN_ERR_UNSUPPORTED: return "unsupported on this device/build";
    case FLUXBIN_ERR_CUDA: return "CUDA error";
    case FLUXBIN_ERR_FORMAT: return "not a packed FluxBin layer";
    }
    return "unknown status";
}

// ---- per-device one-time set-up: SM count, shared-memory opt-in, dynamic-smem base probe --------

namespace {

__device__ uint32_t g_smem_base_probe;

struct DeviceInfo {
    bool ready = false;
    bool ok = false;
    int num_sms = 0;
};
DeviceInfo g_dev[kMaxDevices];
std::mutex g_dev_mutex;

fluxbin_status_t device_setup(int dev, int *num_sms)
{
    if (dev < 0 || dev >= kMaxDevices) return FLUXBIN_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    DeviceInfo &d = g_dev[dev];
    if (!d.ready) {
        int major = 0, sms = 0;
        FB_CUDA(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
        FB_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        d.num_sms = sms;
        d.ok = false;
        if (major == 10) {
            fluxbin_status_t st = fb::opt_in_all_kernels();
            if (st != FLUXBIN_OK) return st;
            FB_CUDA(cudaFuncSetAttribute(fbk::fluxbin_debug_tables_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)fbk::smem_bytes<1>()));
            FB_CUDA(cudaFuncSetAttribute(fbk::fluxbin_smem_base_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)fbk::smem_bytes<1>()));
            // where does dynamic shared memory start?  the tables need the window below 0x10000
            uint32_t *probe = nullptr;
            FB_CUDA(cudaGetSymbolAddress((void **)&probe, g_smem_base_probe));
            fbk::fluxbin_smem_base_kernel<<<1, 32, fbk::smem_bytes<1>(), 0>>>(probe);
            FB_CUDA(cudaGetLastError());
            uint32_t base = 0xffffffffu;
            FB_CUDA(cudaMemcpy(&base, probe, sizeof(base), cudaMemcpyDeviceToHost));
            d.ok = (base <= fbk::kTabBase);
        }
        d.ready = true;
    }
    if (num_sms) *num_sms = d.num_sms;
    return d.ok ? FLUXBIN_OK : FLUXBIN_ERR_UNSUPPORTED;
}

fluxbin_status_t make_handle(const FbHeader &h, void *d_packed, size_t d_bytes, fluxbin_weight_t **out)
{
    if (((uintptr_t)d_packed & 15) != 0) return FLUXBIN_ERR_ALIGNMENT;
    if (d_bytes < h.total_bytes) return FLUXBIN_ERR_BUFFER_TOO_SMALL;
    int dev = 0, sms = 0;
    FB_CUDA(cudaGetDevice(&dev));
    fluxbin_status_t st = device_setup(dev, &sms);
    if (st != FLUXBIN_OK) return st;
    fluxbin_weight_t *w = new (std::nothrow) fluxbin_weight_t;
    if (!w) return FLUXBIN_ERR_UNSUPPORTED;
    w->h = h;
    w->d_packed = d_packed;
    w->d_bytes = d_bytes;
    w->device = dev;
    w->num_sms = sms;
    w->tile_rb = 16;
    if ((h.nrb + w->tile_rb - 1) / w->tile_rb > fbk::kMaxTiles) w->tile_rb = (h.nrb + fbk::kMaxTiles - 1) / fbk::kMaxTiles;
    w->ntiles = (h.nrb + w->tile_rb - 1) / w->tile_rb;
    w->table_format = FLUXBIN_TABLES_FP32;
    for (auto &slot : w->single) slot.store(nullptr);
    *out = w;
    return FLUXBIN_OK;
}

} // namespace

extern "C" fluxbin_status_t fluxbin_pack(const fluxbin_layer_desc_t *desc, void *d_packed, size_t d_bytes,
                                         void *cuda_stream, fluxbin_weight_t **out)
{
    if (!out || !d_packed) return FLUXBIN_ERR_NULL;
    *out = nullptr;
    fluxbin_status_t st = fluxbin_validate(desc);
    if (st != FLUXBIN_OK) return st;
    size_t bytes = fluxbin_packed_size(desc);
    if (bytes == 0) return FLUXBIN_ERR_SHAPE;
    if (d_bytes < bytes) return FLUXBIN_ERR_BUFFER_TOO_SMALL;
    if (((uintptr_t)d_packed & 15) != 0) return FLUXBIN_ERR_ALIGNMENT;
    void *host = std::malloc(bytes);
    if (!host) return FLUXBIN_ERR_UNSUPPORTED;
    st = fluxbin_pack_host(desc, host, bytes);
    if (st == FLUXBIN_OK) {
        FbHeader h;
        std::memcpy(&h, host, sizeof(h));
        cudaStream_t s = (cudaStream_t)cuda_stream;
        cudaError_t e = cudaMemcpyAsync(d_packed, host, bytes, cudaMemcpyHostToDevice, s);
        if (e == cudaSuccess) e = cudaStreamSynchronize(s);
        if (e != cudaSuccess) st = cuda_fail(e);
        else st = make_handle(h, d_packed, d_bytes, out);
    }
    std::free(host);
    return st;
}

extern "C" fluxbin_status_t fluxbin_attach(const void *h_header, size_t header_bytes, void *d_packed, size_t d_bytes,
                                           fluxbin_weight_t **out)
{
    if (!out || !d_packed) return FLUXBIN_ERR_NULL;
    *out = nullptr;
    FbHeader h;
    fluxbin_status_t st = check_header(h_header, header_bytes, h);
    if (st != FLUXBIN_OK) return st;
    return make_handle(h, d_packed, d_bytes, out);
}

extern "C" fluxbin_status_t fluxbin_unpack(const fluxbin_weight_t *w, fluxbin_layer_desc_t *host_out, void *cuda_stream)
{
    if (!w || !host_out) return FLUXBIN_ERR_NULL;
    size_t bytes = (size_t)w->h.total_bytes;
    void *host = std::malloc(bytes);
    if (!host) return FLUXBIN_ERR_UNSUPPORTED;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    cudaError_t e = cudaMemcpyAsync(host, w->d_packed, bytes, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    fluxbin_status_t st = (e == cudaSuccess) ? fluxbin_unpack_host(host, bytes, host_out) : cuda_fail(e);
    std::free(host);
    return st;
}

extern "C" fluxbin_status_t fluxbin_weight_dims(const fluxbin_weight_t *w, fluxbin_layer_desc_t *out)
{
    if (!w || !out) return FLUXBIN_ERR_NULL;
    out->M = w->h.M; out->N = w->h.N; out->Kb = w->h.Kb; out->Ks = w->h.Ks; out->g = w->h.g; out->n_sal = w->h.n_sal;
    return FLUXBIN_OK;
}

extern "C" void fluxbin_free(fluxbin_weight_t *w)
{
    if (!w) return;
    for (auto &slot : w->single) delete slot.load();
    delete w;
}

extern "C" int32_t fluxbin_weight_device(const fluxbin_weight_t *w) { return w ? w->device : -1; }

extern "C" int32_t fluxbin_num_table_sets(const fluxbin_weight_t *w) { return w ? w->h.npairs[0] + w->h.npairs[1] : -1; }

extern "C" fluxbin_status_t fluxbin_set_table_format(fluxbin_weight_t *w, int32_t format)
{
    if (!w) return FLUXBIN_ERR_NULL;
    if (format != FLUXBIN_TABLES_FP32 && format != FLUXBIN_TABLES_FP16 && format != FLUXBIN_TABLES_FP32_MU4) return FLUXBIN_ERR_RANGE;
    // the mu = 4 kernels exist for row-scale groups of a multiple of 128 columns (the configurations of the paper's
    // sub-vector-size study)
    if (format == FLUXBIN_TABLES_FP32_MU4 && w->h.sps[0] != 16) return FLUXBIN_ERR_UNSUPPORTED;
    w->table_format = format;
    return FLUXBIN_OK;
}

extern "C" int32_t fluxbin_get_table_format(const fluxbin_weight_t *w) { return w ? w->table_format : -1; }

// Batch vectors per launch: B is processed in chunks of up to four (fp32 table entries) or eight (fp16
// entries).  A chunk runs the kernel whose table entries hold its vectors side by side in 4, 8 or 16 bytes
// (LDS.32 / .64 / .128): the weights stream once per chunk and one address computation serves the whole
// entry.  A single vector always uses fp32 entries (nothing to share a word with).
static int chunk_size(int fmt) { return fmt == FLUXBIN_TABLES_FP16 ? 8 : 4; }
static int nvec_for(int nb) { return nb == 1 ? 1 : nb == 2 ? 2 : nb <= 4 ? 4 : 8; }
static int mode_for(int nb, int fmt)
{
    if (fmt == FLUXBIN_TABLES_FP32_MU4) return 32 + nvec_for(nb);
    return (fmt == FLUXBIN_TABLES_FP16 && nb >= 2) ? 16 + nvec_for(nb) : nvec_for(nb);
}
static int ws_bt(int B, int fmt) { return nvec_for(B < chunk_size(fmt) ? B : chunk_size(fmt)); }   // accumulator rows per layer

// The chunks of a batch of B vectors, largest first: full chunks, then the rest.  A rest that would run with
// dead vectors in its entries (3 with fp32 entries; 5 or 6 with fp16 entries) is cut once more (2 + 1, 4 + 1,
// 4 + 2) when the launch streams enough weight bytes for the second pass to cost less than the dead vectors do
// (measured on a 16-layer 70B-shaped stack: 12 %, 16 % and 11 % faster; an extra launch costs a few microseconds,
// about what 32 MB of weights take).
constexpr long long kSplitRestBytes = 128ll << 20;
struct Chunks {
    int n = 0;
    int nb[4] = {0, 0, 0, 0};       // sizes of the chunks after the full ones
    int full = 0;                   // number of full chunks (of chunk_size vectors)
    int rest_n = 0;
};
static Chunks chunks_of(int B, int fmt, long long weight_bytes)
{
    Chunks c;
    const int CH = chunk_size(fmt);
    c.full = B / CH;
    const int r = B % CH;
    const bool big = weight_bytes >= kSplitRestBytes;
    if (r > 0) {
        int first = r;
        if (big && fmt != FLUXBIN_TABLES_FP16 && r == 3) first = 2;
        if (big && fmt == FLUXBIN_TABLES_FP16 && (r == 5 || r == 6)) first = 4;
        c.nb[c.rest_n++] = first;
        if (first < r) c.nb[c.rest_n++] = r - first;
    }
    c.n = c.full + c.rest_n;
    return c;
}
// size and first vector of chunk i
static int chunk_nb(const Chunks &c, int fmt, int i) { return i < c.full ? chunk_size(fmt) : c.nb[i - c.full]; }
static int chunk_begin(const Chunks &c, int fmt, int i)
{
    int b = (i < c.full ? i : c.full) * chunk_size(fmt);
    for (int j = c.full; j < i; ++j) b += c.nb[j - c.full];
    return b;
}

extern "C" int32_t fluxbin_num_launches(const fluxbin_weight_t *w, int32_t B)
{
    if (!w || B < 1) return -1;
    return chunks_of(B, w->table_format, (long long)w->h.total_bytes).n;
}

// ---- workspace ----------------------------------------------------------------------------------

static size_t acc_bytes(const fluxbin_weight_t *w, int bt) { return ((size_t)bt * w->h.Mpad * 4 + 255) / 256 * 256; }

extern "C" size_t fluxbin_workspace_size(const fluxbin_weight_t *w, int32_t B)
{
    if (!w || B < 1) return 0;
    int bt = ws_bt(B, w->table_format);
    return acc_bytes(w, bt) + ((size_t)w->ntiles * 4 + 255) / 256 * 256 + 256;    // + the launch counters
}

extern "C" fluxbin_status_t fluxbin_workspace_init(void *d_workspace, size_t bytes, void *cuda_stream)
{
    if (!d_workspace) return FLUXBIN_ERR_NULL;
    FB_CUDA(cudaMemsetAsync(d_workspace, 0, bytes, (cudaStream_t)cuda_stream));
    return FLUXBIN_OK;
}

// ---- the layer ------------------------------------------------------------------------------------

// The kernel instantiation for a launch mode (1, 2, 4 vectors with fp32 tables, 16 + (2, 4, 8) with fp16 tables,
// 32 + (1, 2, 4) with fp32 tables of mu = 4 sub-vectors), a row-scale format class (sub-vectors per scale segment of the global / salient region) and the number of
// pairs walked per row block (2 exists for the modes with 4-byte table entries: 1 and 16 + 2).
template <int S0, int S1, int BT> static const void *kernel_of(int np)
{
    if constexpr (fbk::geom(BT) == 1 && !fbk::mu4(BT)) {
        if (np == 2) return (const void *)fbk::fluxbin_linear_kernel<S0, S1, BT, 2>;
    }
    return (const void *)fbk::fluxbin_linear_kernel<S0, S1, BT, 1>;
}
template <int BT> static const void *kernel_of_bt(int s0, int s1, int np)
{
    if (s0 == 16 && s1 == 16) return kernel_of<16, 16, BT>(np);
    if (s0 == 16) return kernel_of<16, 1, BT>(np);
    if (s0 == 8) return kernel_of<8, 1, BT>(np);
    return kernel_of<4, 1, BT>(np);
}
template <int BT> static const void *kernel_of_mu4(int s0, int s1)
{
    if (s0 == 16 && s1 == 16) return kernel_of<16, 16, BT>(1);
    if (s0 == 16) return kernel_of<16, 1, BT>(1);
    return nullptr;                     // fluxbin_set_table_format refuses the other classes
}
static const void *kernel_for(int mode, int s0, int s1, int np)
{
    switch (mode) {
    case 32 + 1: return kernel_of_mu4<32 + 1>(s0, s1);
    case 32 + 2: return kernel_of_mu4<32 + 2>(s0, s1);
    case 32 + 4: return kernel_of_mu4<32 + 4>(s0, s1);
    case 1: return kernel_of_bt<1>(s0, s1, np);
    case 2: return kernel_of_bt<2>(s0, s1, np);
    case 4: return kernel_of_bt<4>(s0, s1, np);
    case 16 + 2: return kernel_of_bt<16 + 2>(s0, s1, np);
    case 16 + 4: return kernel_of_bt<16 + 4>(s0, s1, np);
    case 16 + 8: return kernel_of_bt<16 + 8>(s0, s1, np);
    }
    return nullptr;
}
constexpr int kNumModes = 9;
static int mode_index(int mode)
{
    if (mode >= 32) return mode == 32 + 1 ? 6 : mode == 32 + 2 ? 7 : 8;
    return mode == 1 ? 0 : mode == 2 ? 1 : mode == 4 ? 2 : mode == 16 + 2 ? 3 : mode == 16 + 4 ? 4 : 5;
}
static int class_index(int s0, int s1) { return (s0 == 16 && s1 == 16) ? 0 : s0 == 16 ? 1 : s0 == 8 ? 2 : 3; }
static int threads_for(int mode) { return fbk::geom(mode) == 4 ? 512 : 256; }
static size_t smem_for(int mode)      // the scratch beside the tables grows with the vectors of the mode
{
    switch (mode) {
    case 1: return fbk::smem_bytes<1>();
    case 2: return fbk::smem_bytes<2>();
    case 4: return fbk::smem_bytes<4>();
    case 16 + 2: return fbk::smem_bytes<16 + 2>();
    case 16 + 4: return fbk::smem_bytes<16 + 4>();
    case 16 + 8: return fbk::smem_bytes<16 + 8>();
    case 32 + 1: return fbk::smem_bytes<32 + 1>();
    case 32 + 2: return fbk::smem_bytes<32 + 2>();
    case 32 + 4: return fbk::smem_bytes<32 + 4>();
    }
    return 0;
}

fluxbin_status_t fb::opt_in_all_kernels()
{
    static const int modes[kNumModes] = {1, 2, 4, 16 + 2, 16 + 4, 16 + 8, 32 + 1, 32 + 2, 32 + 4};
    static const int cls[4][2] = {{16, 16}, {16, 1}, {8, 1}, {4, 1}};
    for (int m : modes)
        for (auto &c : cls)
            for (int np = 1; np <= ((fbk::geom(m) == 1 && !fbk::mu4(m)) ? 2 : 1); ++np) {
                const void *k = kernel_for(m, c[0], c[1], np);
                if (k) FB_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_for(m)));
            }
    return FLUXBIN_OK;
}

// Work-split cost model, measured on B200 in units of half a 1152-byte item (about 50 ns per CTA):
// an item with one row scale per sub-vector (3072 bytes) takes about 2x a plain item; building one
// table set (two dependent loads, 8K table entries, two barriers) takes about as long as 22 items
// (re-measured against the current row loop: 28 / 36 / 44 / 56 -> 5.61 / 5.80 / 5.85 / 5.83 TB/s on the stack plan).
constexpr int kBuildCost = 44;
// With four or eight vectors in fp16 table entries an item takes about half the time it takes with fp32 entries,
// a build (more vectors per entry, conversions) does not: measured 44 / 66 / 88 / 132 -> 3.29 / 3.47 / 3.51 / 3.46
// TB/s at batch 4 and 1.73 / 1.81 / 1.81 / 1.81 at batch 8.  (With fp32 entries, batch 2 and 4: no effect.)
constexpr int kBuildCostHalfWide = 88;
// mu = 4: a table set has 32 rows of entries instead of 256 and an item twice the lookups, so a build is worth far
// fewer items (the dependent loads and the two barriers remain).
constexpr int kBuildCostMu4 = 12;
static int build_cost_for(int mode)
{
    if (fbk::mu4(mode)) return kBuildCostMu4;
    return (mode == 16 + 4 || mode == 16 + 8) ? kBuildCostHalfWide : kBuildCost;    // two vectors in fp16 entries: 36 / 44 / 56 / 66 all within 1 %
}
// The reduction epilogue a CTA runs when it leaves an entry (fence, tickets, read-back of the tiles it
// completed): a fixed part plus a part that grows with the rows to convert.
static long long epilogue_cost(const FbHeader &h) { return 80 + h.Mpad / 128; }

static long long couple_cost_of(const FbHeader &h)
{
    if (h.npairs[0] < 2 || (h.npairs[0] & 1)) return 0;
    return 2 * (kBuildCost + (long long)h.nrb * 2);
}

static void item_costs(int sps0, int sps1, int cost[2])
{
    cost[0] = 2;
    cost[1] = (sps1 == sps0) ? 2 : 4;
}

// An item of a narrow last salient pair (8 or 16 steps instead of 32) is costed like a full one: the loop for items
// with one scale per sub-vector keeps a single item in flight per warp (a full one fills 24 registers), so an item
// takes a load latency whatever its size.  (Measured: costing it by its bytes left the CTAs that own the narrow
// pair with twice the items and made one-launch-per-group runs 5 % slower; a two-deep loop for the narrow items
// cost the whole kernel spills.)
static int last_salient_item_cost(const FbHeader &h, int cost1)
{
    (void)h;
    return cost1;
}

static long long entry_cost(const FbHeader &h, int sps1, int build_cost)
{
    int c[2];
    item_costs(h.sps[0], sps1, c);
    long long cost = (long long)h.npairs[0] * (build_cost + (long long)h.nrb * c[0]) + epilogue_cost(h);
    if (h.npairs[1] > 0)
        cost += (long long)(h.npairs[1] - 1) * (build_cost + (long long)h.nrb * c[1]) +
                (build_cost + (long long)h.nrb * last_salient_item_cost(h, c[1]));
    return cost;
}

// The two-pairs-per-row-block kernel pays two table builds per run of rows but has the better row loop (one
// reduction per two items, loads requested half an item earlier).  Measured on B200 (batch 1) against the one-pair
// kernel with its first item in flight during the build: it wins once a CTA's share is worth about 200 to 270 plain
// items (cost 400 to 540: the {gate, up} launch of a 70B-shaped layer, one launch per layer, one plan for a stack)
// and loses below that -- with the threshold at 60 instead of 400 the 7B-shaped set ran 7 % slower with one launch
// per dependency group (5.43 against 5.05 us per linear), the 13B-shaped set 5 %, the 70B-shaped layers 2 %; with
// it at 1000 the 70B-shaped groups lose 1.4 %, at 3000 one launch per layer loses 7 %.
constexpr long long kCoupleMinShare = 400;

// How a launch is cut: grid size, the statically dealt part of the cost line, the number of shares, and
// how many pairs the kernel walks per row block (2: the two-pairs-per-row-block kernel).
struct LaunchShape {
    int grid, nshares, np;
    long long static_cost;
};

static cudaError_t launch_shape(int dev, int mode, int s0, int s1, long long total_cost, int num_sms, long long items,
                                long long couple_cost, bool allow_dynamic, LaunchShape *out)
{
    // resident CTAs per SM of an instantiation, per device (0 = not asked yet; racing threads store the same value)
    static std::atomic<int> occ_of[kMaxDevices][kNumModes][4];
    std::atomic<int> &slot = occ_of[dev][mode_index(mode)][class_index(s0, s1)];
    int occ = slot.load(std::memory_order_relaxed);
    if (occ == 0) {
        int o = 0;
        cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o, kernel_for(mode, s0, s1, 1), threads_for(mode), smem_for(mode));
        if (e != cudaSuccess) return e;
        occ = o > 0 ? o : 1;
        slot.store(occ, std::memory_order_relaxed);
    }
    long long grid = (long long)num_sms * occ;
    if (items < grid) grid = items;
    if (grid > kMaxGrid) grid = kMaxGrid;
    if (!allow_dynamic && grid > fbk::kMaxSingleShares) grid = fbk::kMaxSingleShares;
    // Launches with enough work deal 90 % of it out statically and cut the rest into three small
    // shares per CTA (each worth >= ~200 items), drawn dynamically; small launches stay static.
    constexpr int dyn_pct = 10, dyn_k = 3;
    const long long rest = total_cost * dyn_pct / 100;
    if (allow_dynamic && rest / (grid * dyn_k) >= 400) {
        out->static_cost = total_cost - rest;
        out->nshares = (int)(grid * (1 + dyn_k));
    } else {
        out->static_cost = total_cost;
        out->nshares = (int)grid;
    }
    out->grid = (int)grid;
    // two pairs per row block when every layer allows it (couple_cost > 0: even pair counts everywhere) and a
    // CTA's share is large enough to pay for the second table build
    out->np = (fbk::geom(mode) == 1 && !fbk::mu4(mode) && couple_cost > 0 && out->static_cost / grid >= kCoupleMinShare) ? 2 : 1;
    return cudaSuccess;
}

// ---- cutting the cost line (host) --------------------------------------------------------------------
// Every pair of an entry costs build_cost + nrb * item_cost of its region, the entry ends with its epilogue
// cost; the entries of a launch lie one after the other.  Share s owns the work items whose start lies in its
// piece [lo, hi) of the line; a cut inside the build part of a work pair goes to its first row block.

struct CutModel {
    int np, build_cost, item_cost[2];
};

// first work item of header h at or after position pos of its own cost line (0 .. all items)
static int first_item_at(const FbHeader &h, const CutModel &m, long long pos)
{
    const int np = m.np;
    const long long w0 = m.item_cost[0], w1 = m.item_cost[1];
    const int wp0 = h.npairs[0] / np;
    const int I0 = wp0 * h.nrb, I1 = h.npairs[1] * h.nrb;
    const long long w1l = last_salient_item_cost(h, m.item_cost[1]);
    const long long Pc0 = np * (m.build_cost + (long long)h.nrb * w0), Pc1 = m.build_cost + (long long)h.nrb * w1;
    const long long Pc1l = m.build_cost + (long long)h.nrb * w1l;
    const long long T0 = (long long)wp0 * Pc0, T1 = h.npairs[1] > 0 ? (long long)(h.npairs[1] - 1) * Pc1 : 0;
    const long long T = T0 + (h.npairs[1] > 0 ? T1 + Pc1l : 0);
    if (pos <= 0) return 0;
    if (pos >= T) return I0 + I1;
    const bool reg1 = pos >= T0;
    const bool last1 = reg1 && pos - T0 >= T1;          // inside the last salient pair (its items may be cheaper)
    const long long rel = reg1 ? pos - T0 : pos, Pc = reg1 ? Pc1 : Pc0, w = last1 ? w1l : reg1 ? w1 : np * w0;
    const long long pair = last1 ? h.npairs[1] - 1 : rel / Pc;
    const long long within = rel - (last1 ? T1 : pair * Pc) - (reg1 ? 1 : np) * m.build_cost;
    long long rb = within <= 0 ? 0 : (within + w - 1) / w;
    if (rb > h.nrb) rb = h.nrb;
    return (reg1 ? I0 : 0) + (int)(pair * h.nrb + rb);
}

static int work_items_of(const FbHeader &h, int np) { return (h.npairs[0] / np + h.npairs[1]) * h.nrb; }

// cuts[s] for s = 0 .. nshares: where share s begins ({n, 0} = the end of the launch).  cost_begin[e] = summed
// cost of the entries before e, cost_begin[n] = the total.
static void cut_launch(const FbHeader *const *hs, const long long *cost_begin, int n, const CutModel &m,
                       const LaunchShape &shape, fbk::ShareCut *cuts)
{
    const long long total = cost_begin[n], rest = total - shape.static_cost;
    const int G = shape.grid, nj = shape.nshares - G;
    int e = 0;
    for (int s = 0; s <= shape.nshares; ++s) {
        long long lo;
        if (s <= G) lo = shape.static_cost * (long long)s / G;
        else lo = shape.static_cost + rest * (long long)(s - G) / nj;
        if (s == shape.nshares) lo = total;
        while (e + 1 < n && cost_begin[e + 1] <= lo) ++e;     // last entry that begins at or before lo
        int item = first_item_at(*hs[e], m, lo - cost_begin[e]);
        int ce = e;
        if (item >= work_items_of(*hs[e], m.np)) { ce = e + 1; item = 0; }
        cuts[s].entry = ce;
        cuts[s].item = item;
    }
    cuts[shape.nshares].entry = n;
    cuts[shape.nshares].item = 0;
}

// Test hook (host only, no GPU): the share bounds of a launch of n packed layers, given their 256-byte headers.
extern "C" fluxbin_status_t fluxbin_debug_cut_shares(int32_t n, const void *const *h_headers, int32_t mode, int32_t pairs_per_row_block,
                                                     int32_t grid, int32_t nshares, int32_t static_percent, int32_t *out_cuts,
                                                     int32_t *out_work_items)
{
    if (!h_headers || !out_cuts) return FLUXBIN_ERR_NULL;
    if (n < 1 || grid < 1 || nshares < grid || static_percent < 1 || static_percent > 100 || (nshares > grid && static_percent == 100))
        return FLUXBIN_ERR_RANGE;
    if (!kernel_for(mode, 16, 1, 1) || pairs_per_row_block < 1 || pairs_per_row_block > 2) return FLUXBIN_ERR_RANGE;
    std::vector<FbHeader> H((size_t)n);
    std::vector<const FbHeader *> hs((size_t)n);
    int sps1 = 0;
    for (int i = 0; i < n; ++i) {
        fluxbin_status_t st = check_header(h_headers[i], FB_HEADER_BYTES, H[(size_t)i]);
        if (st != FLUXBIN_OK) return st;
        hs[(size_t)i] = &H[(size_t)i];
        if (H[(size_t)i].npairs[1] > 0) sps1 = H[(size_t)i].sps[1];
        if (pairs_per_row_block == 2 && (H[(size_t)i].npairs[0] & 1)) return FLUXBIN_ERR_UNSUPPORTED;
    }
    if (sps1 == 0) sps1 = 1;
    CutModel m;
    m.np = pairs_per_row_block;
    m.build_cost = build_cost_for(mode);
    item_costs(H[0].sps[0], sps1, m.item_cost);
    std::vector<long long> cost_begin((size_t)n + 1);
    long long cost = 0;
    for (int i = 0; i < n; ++i) {
        cost_begin[(size_t)i] = cost;
        cost += entry_cost(H[(size_t)i], sps1, m.build_cost);
        if (out_work_items) out_work_items[i] = work_items_of(H[(size_t)i], m.np);
    }
    cost_begin[(size_t)n] = cost;
    LaunchShape shape;
    shape.grid = grid; shape.nshares = nshares; shape.np = m.np;
    shape.static_cost = nshares > grid ? cost * static_percent / 100 : cost;
    std::vector<fbk::ShareCut> cuts((size_t)nshares + 1);
    cut_launch(hs.data(), cost_begin.data(), n, m, shape, cuts.data());
    for (int s = 0; s <= nshares; ++s) { out_cuts[2 * s] = cuts[(size_t)s].entry; out_cuts[2 * s + 1] = cuts[(size_t)s].item; }
    return FLUXBIN_OK;
}

static cudaError_t launch_kernel(int mode, int s0, int s1, const LaunchShape &shape, const fbk::LaunchParams &p, cudaStream_t s)
{
    // launched with programmatic stream serialization: the kernel may start while its predecessor in
    // the stream drains (it waits inside, before touching activations or workspace)
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)shape.grid);
    cfg.blockDim = dim3((unsigned)threads_for(mode));
    cfg.dynamicSmemBytes = smem_for(mode);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
#ifdef FB_TRACE
    static std::atomic<int> launches{0};
    const_cast<fbk::LaunchParams &>(p).trace_slot = launches.fetch_add(1) & 7;
#endif
    void *args[1] = {(void *)&p};
    return cudaLaunchKernelExC(&cfg, kernel_for(mode, s0, s1, shape.np), args);
}

static void fill_entry(fbk::LinearEntry &E, const fluxbin_weight_t *w, const uint16_t *x, int64_t ldx, void *y, int64_t ldy,
                       float *acc, unsigned *tickets)
{
    E.packed = (const uint8_t *)w->d_packed;
    E.x = x; E.y = y; E.acc = acc; E.tickets = tickets;
    E.ldx = ldx; E.ldy = ldy; E.acc2 = nullptr;
    E.off_coldesc = w->h.off_coldesc; E.off_items[0] = w->h.off_items[0]; E.off_items[1] = w->h.off_items[1];
    E.M = w->h.M; E.N = w->h.N; E.Kb = w->h.Kb; E.nrb = w->h.nrb;
    E.npairs[0] = w->h.npairs[0]; E.npairs[1] = w->h.npairs[1];
    E.arrivals = w->h.npairs[0] + w->h.npairs[1];
    E.tile_rb = w->tile_rb; E.ntiles = w->ntiles; E.flags = w->h.sal_last_w;
}

// The launch shape and the share bounds of a one-layer launch in a given mode depend on the layer alone: they are
// worked out on first use and kept with the handle.
static const SingleLaunch *single_launch_of(const fluxbin_weight_t *w, int mode, cudaError_t *err)
{
    std::atomic<SingleLaunch *> &slot = w->single[mode_index(mode)];
    SingleLaunch *sl = slot.load(std::memory_order_acquire);
    if (sl) return sl;
    const int s0 = w->h.sps[0], s1 = w->h.npairs[1] > 0 ? w->h.sps[1] : 1;
    CutModel m;
    m.build_cost = build_cost_for(mode);
    item_costs(s0, s1, m.item_cost);
    const long long total = entry_cost(w->h, s1, m.build_cost);
    const long long items = (long long)(w->h.npairs[0] + w->h.npairs[1]) * w->h.nrb;
    LaunchShape shape;
    *err = launch_shape(w->device, mode, s0, s1, total, w->num_sms, items, couple_cost_of(w->h), false, &shape);
    if (*err != cudaSuccess) return nullptr;
    m.np = shape.np;
    sl = new (std::nothrow) SingleLaunch;
    if (!sl) { *err = cudaErrorMemoryAllocation; return nullptr; }
    sl->grid = shape.grid; sl->np = shape.np;
    std::vector<fbk::ShareCut> cuts((size_t)shape.nshares + 1);
    const FbHeader *hs[1] = {&w->h};
    const long long cb[2] = {0, total};
    cut_launch(hs, cb, 1, m, shape, cuts.data());
    const int all = work_items_of(w->h, m.np);
    for (int s = 0; s <= shape.nshares; ++s) sl->cut[s] = cuts[s].entry >= 1 ? all : cuts[s].item;
    SingleLaunch *expected = nullptr;
    if (!slot.compare_exchange_strong(expected, sl, std::memory_order_acq_rel)) { delete sl; sl = expected; }
    return sl;
}

extern "C" fluxbin_status_t fluxbin_linear(const fluxbin_weight_t *w, const uint16_t *d_x, int32_t B, int64_t ldx,
                                           void *d_y, int32_t y_is_fp32, int64_t ldy,
                                           void *d_workspace, size_t ws_bytes, void *cuda_stream)
{
    if (!w || !d_x || !d_y || !d_workspace) return FLUXBIN_ERR_NULL;
    if (B < 1 || ldx < w->h.N || ldy < w->h.M) return FLUXBIN_ERR_RANGE;
    if ((((uintptr_t)d_x) & 15) || (((uintptr_t)d_y) & 15) || (((uintptr_t)d_workspace) & 15)) return FLUXBIN_ERR_ALIGNMENT;
    if (ws_bytes < fluxbin_workspace_size(w, B)) return FLUXBIN_ERR_BUFFER_TOO_SMALL;
    // a 16-segment salient region only exists with a single scale group, where sps[0] is 16 too
    if (w->h.npairs[1] > 0 && w->h.sps[1] == 16 && w->h.sps[0] != 16) return FLUXBIN_ERR_FORMAT;
    int dev = -1;
    FB_CUDA(cudaGetDevice(&dev));
    if (dev != w->device) return FLUXBIN_ERR_UNSUPPORTED;      // the layer lives on another device than the current one
    cudaStream_t s = (cudaStream_t)cuda_stream;

    fbk::LaunchParams p;
    p.table = nullptr;
    p.cuts = nullptr;
    p.n = 1;
    p.y_fp32 = y_is_fp32 != 0;
    const int fmt = w->table_format;
    const int bt_ws = ws_bt(B, fmt);
    float *acc = (float *)d_workspace;
    unsigned *tickets = (unsigned *)((uint8_t *)d_workspace + acc_bytes(w, bt_ws));
    p.counters = (unsigned *)((uint8_t *)d_workspace + acc_bytes(w, bt_ws) + ((size_t)w->ntiles * 4 + 255) / 256 * 256);
    const int s0 = w->h.sps[0], s1 = w->h.npairs[1] > 0 ? w->h.sps[1] : 1;

    const size_t ysz = y_is_fp32 ? 4 : 2;
    const Chunks ch = chunks_of(B, fmt, (long long)w->h.total_bytes);
    for (int c = 0; c < ch.n; ++c) {
        const int nb = chunk_nb(ch, fmt, c), b0 = chunk_begin(ch, fmt, c);
        const int mode = mode_for(nb, fmt);
        cudaError_t e = cudaSuccess;
        const SingleLaunch *sl = single_launch_of(w, mode, &e);
        if (!sl) return cuda_fail(e);
        fill_entry(p.single, w, d_x + (int64_t)b0 * ldx, ldx, (uint8_t *)d_y + (size_t)b0 * ldy * ysz, ldy, acc, tickets);
        p.nb = nb;
        p.nshares = sl->grid;
        std::memcpy(p.single_cut, sl->cut, sizeof(int) * ((size_t)sl->grid + 1));
        LaunchShape shape;
        shape.grid = sl->grid; shape.nshares = sl->grid; shape.np = sl->np; shape.static_cost = 0;
        e = launch_kernel(mode, s0, s1, shape, p, s);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    return FLUXBIN_OK;
}

// ---- plans: many layers in one persistent launch -------------------------------------------------

struct PlanChunk {
    int nb, mode;
    LaunchShape shape;
    const fbk::LinearEntry *d_entries;
    const fbk::ShareCut *d_cuts;
};

struct fluxbin_plan {
    int n, B, y_fp32, table_format, device;
    int sps0, sps1;
    std::vector<PlanChunk> chunks;
    unsigned *d_counters;
};

static size_t entry_ws_bytes(const fluxbin_weight_t *w, int bt)
{
    return acc_bytes(w, bt) + ((size_t)w->ntiles * 4 + 255) / 256 * 256;
}

// device table of one chunk: the entries, then the share cuts (at most 4 shares per CTA of the largest grid)
static size_t chunk_table_bytes(int n)
{
    return ((size_t)n * sizeof(fbk::LinearEntry) + ((size_t)4 * kMaxGrid + 1) * sizeof(fbk::ShareCut) + 255) / 256 * 256;
}

extern "C" size_t fluxbin_plan_table_bytes(int32_t n, int32_t B)
{
    if (n < 1 || B < 1) return 0;
    // an upper bound over the table formats and the cut of the rest
    const int most = chunks_of(B, FLUXBIN_TABLES_FP32, kSplitRestBytes).n;
    return chunk_table_bytes(n) * (size_t)most;
}

extern "C" size_t fluxbin_plan_workspace_bytes(int32_t n, const fluxbin_weight_t *const *w, int32_t B)
{
    if (n < 1 || B < 1 || !w) return 0;
    if (!w[0]) return 0;
    const int bt = ws_bt(B, w[0]->table_format);
    size_t total = 0;
    for (int i = 0; i < n; ++i) {
        if (!w[i]) return 0;
        total += entry_ws_bytes(w[i], bt);
    }
    return total + 256;      // + the launch counters
}

// gate_up: n_gated pairs {gate member, up member} whose outputs are combined as silu(gate) * up into the gate's y
static fluxbin_status_t plan_create_impl(int32_t n, const fluxbin_weight_t *const *w,
                                         const uint16_t *const *d_x, const int64_t *ldx,
                                         void *const *d_y, const int64_t *ldy,
                                         const int32_t *gate_up, int32_t n_gated,
                                         int32_t B, int32_t y_is_fp32,
                                         void *d_table, size_t table_bytes,
                                         void *d_workspace, size_t ws_bytes,
                                         void *cuda_stream, fluxbin_plan_t **out)
{
    if (!out) return FLUXBIN_ERR_NULL;
    *out = nullptr;
    if (!w || !d_x || !ldx || !d_y || !ldy || !d_table || !d_workspace) return FLUXBIN_ERR_NULL;
    if (n < 1 || B < 1 || n_gated < 0 || (n_gated > 0 && !gate_up)) return n_gated > 0 && !gate_up ? FLUXBIN_ERR_NULL : FLUXBIN_ERR_RANGE;
    std::vector<int> role((size_t)n, 0), partner((size_t)n, -1);
    for (int p = 0; p < n_gated; ++p) {
        const int g = gate_up[2 * p], u = gate_up[2 * p + 1];
        if (g < 0 || g >= n || u < 0 || u >= n || g == u) return FLUXBIN_ERR_RANGE;
        if (role[(size_t)g] || role[(size_t)u]) return FLUXBIN_ERR_RANGE;          // a member belongs to at most one pair
        if (!w[g] || !w[u]) return FLUXBIN_ERR_NULL;
        if (w[g]->h.M != w[u]->h.M) return FLUXBIN_ERR_SHAPE;                     // the two outputs are multiplied row by row
        role[(size_t)g] = 1; role[(size_t)u] = 2;
        partner[(size_t)g] = u; partner[(size_t)u] = g;
    }
    if ((((uintptr_t)d_table) & 15) || (((uintptr_t)d_workspace) & 15)) return FLUXBIN_ERR_ALIGNMENT;
    if (table_bytes < fluxbin_plan_table_bytes(n, B)) return FLUXBIN_ERR_BUFFER_TOO_SMALL;
    int sps1 = 0;
    for (int i = 0; i < n; ++i) {
        const bool has_y = role[(size_t)i] != 2;              // the up member of a gated pair writes into the gate's y
        if (!w[i] || !d_x[i] || (has_y && !d_y[i])) return FLUXBIN_ERR_NULL;
        if (ldx[i] < w[i]->h.N || (has_y && ldy[i] < w[i]->h.M)) return FLUXBIN_ERR_RANGE;
        if ((((uintptr_t)d_x[i]) & 15) || (has_y && (((uintptr_t)d_y[i]) & 15))) return FLUXBIN_ERR_ALIGNMENT;
        if (w[i]->device != w[0]->device) return FLUXBIN_ERR_UNSUPPORTED;      // all members on one device
        if (w[i]->h.sps[0] != w[0]->h.sps[0]) return FLUXBIN_ERR_UNSUPPORTED;
        if (w[i]->table_format != w[0]->table_format) return FLUXBIN_ERR_UNSUPPORTED;
        if (w[i]->h.npairs[1] > 0) {          // the salient format only matters where there is a salient region
            if (w[i]->h.sps[1] == 16 && w[i]->h.sps[0] != 16) return FLUXBIN_ERR_FORMAT;
            if (sps1 != 0 && w[i]->h.sps[1] != sps1) return FLUXBIN_ERR_UNSUPPORTED;
            sps1 = w[i]->h.sps[1];
        }
    }
    if (sps1 == 0) sps1 = 1;
    if (ws_bytes < fluxbin_plan_workspace_bytes(n, w, B)) return FLUXBIN_ERR_BUFFER_TOO_SMALL;
    int dev = -1;
    FB_CUDA(cudaGetDevice(&dev));
    if (dev != w[0]->device) return FLUXBIN_ERR_UNSUPPORTED;       // create (and run) the plan with the layers' device current

    const int fmt = w[0]->table_format, sps0 = w[0]->h.sps[0];
    long long weight_bytes = 0, items = 0, couple_cost = 0;
    bool all_even = true;
    std::vector<const FbHeader *> hs((size_t)n);
    for (int i = 0; i < n; ++i) {
        weight_bytes += (long long)w[i]->h.total_bytes;
        items += (long long)(w[i]->h.npairs[0] + w[i]->h.npairs[1]) * w[i]->h.nrb;
        const long long c = couple_cost_of(w[i]->h);
        if (c == 0) all_even = false;
        if (c > couple_cost) couple_cost = c;
        hs[(size_t)i] = &w[i]->h;
    }
    if (!all_even) couple_cost = 0;
    const Chunks ch = chunks_of(B, fmt, weight_bytes);
    const int nchunks = ch.n, bt = ws_bt(B, fmt);
    const size_t ysz = y_is_fp32 ? 4 : 2;
    const size_t ctb = chunk_table_bytes(n);
    std::vector<uint8_t> host(ctb * (size_t)nchunks, 0);
    fluxbin_plan *p = new (std::nothrow) fluxbin_plan;
    if (!p) return FLUXBIN_ERR_UNSUPPORTED;
    std::vector<long long> cost_begin((size_t)n + 1);
    for (int c = 0; c < nchunks; ++c) {
        uint8_t *ws = (uint8_t *)d_workspace;
        PlanChunk pc;
        pc.nb = chunk_nb(ch, fmt, c);
        pc.mode = mode_for(pc.nb, fmt);
        const int b0 = chunk_begin(ch, fmt, c);
        CutModel m;
        m.build_cost = build_cost_for(pc.mode);
        item_costs(sps0, sps1, m.item_cost);
        fbk::LinearEntry *entries = (fbk::LinearEntry *)(host.data() + ctb * (size_t)c);
        long long cost = 0;
        for (int i = 0; i < n; ++i) {
            float *acc = (float *)ws;
            unsigned *tickets = (unsigned *)(ws + acc_bytes(w[i], bt));
            const int yi = role[(size_t)i] == 2 ? partner[(size_t)i] : i;      // whose output buffer this member writes
            fill_entry(entries[i], w[i], d_x[i] + (int64_t)b0 * ldx[i], ldx[i], (uint8_t *)d_y[yi] + (size_t)b0 * ldy[yi] * ysz,
                       ldy[yi], acc, tickets);
            cost_begin[(size_t)i] = cost;
            cost += entry_cost(w[i]->h, sps1, m.build_cost);
            ws += entry_ws_bytes(w[i], bt);
        }
        cost_begin[(size_t)n] = cost;
        for (int i = 0; i < n; ++i) {
            if (!role[(size_t)i]) continue;
            // the two layers of a gated pair count their arrivals on one set of tickets (the gate's) and see each
            // other's accumulators: whoever completes a row tile of both writes silu(gate) * up
            const int j = partner[(size_t)i], g = role[(size_t)i] == 1 ? i : j;
            entries[i].acc2 = entries[j].acc;
            entries[i].tickets = entries[g].tickets;
            entries[i].arrivals = w[i]->h.npairs[0] + w[i]->h.npairs[1] + w[j]->h.npairs[0] + w[j]->h.npairs[1];
            entries[i].flags |= role[(size_t)i] << 8;
        }
        cudaError_t e = launch_shape(dev, pc.mode, sps0, sps1, cost, w[0]->num_sms, items, couple_cost, true, &pc.shape);
        if (e != cudaSuccess) { delete p; return cuda_fail(e); }
        m.np = pc.shape.np;
        fbk::ShareCut *cuts = (fbk::ShareCut *)(entries + n);
        cut_launch(hs.data(), cost_begin.data(), n, m, pc.shape, cuts);
        pc.d_entries = (const fbk::LinearEntry *)((uint8_t *)d_table + ctb * (size_t)c);
        pc.d_cuts = (const fbk::ShareCut *)(pc.d_entries + n);
        p->chunks.push_back(pc);
    }
    cudaStream_t s = (cudaStream_t)cuda_stream;
    cudaError_t e = cudaMemcpyAsync(d_table, host.data(), host.size(), cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) { delete p; return cuda_fail(e); }

    p->n = n; p->B = B; p->y_fp32 = y_is_fp32 != 0; p->table_format = fmt; p->device = dev;
    p->sps0 = sps0; p->sps1 = sps1;
    p->d_counters = (unsigned *)((uint8_t *)d_workspace + fluxbin_plan_workspace_bytes(n, w, B) - 256);
    *out = p;
    return FLUXBIN_OK;
}

extern "C" fluxbin_status_t fluxbin_plan_create(int32_t n, const fluxbin_weight_t *const *w,
                                                const uint16_t *const *d_x, const int64_t *ldx,
                                                void *const *d_y, const int64_t *ldy,
                                                int32_t B, int32_t y_is_fp32,
                                                void *d_table, size_t table_bytes,
                                                void *d_workspace, size_t ws_bytes,
                                                void *cuda_stream, fluxbin_plan_t **out)
{
    return plan_create_impl(n, w, d_x, ldx, d_y, ldy, nullptr, 0, B, y_is_fp32, d_table, table_bytes, d_workspace, ws_bytes,
                            cuda_stream, out);
}

extern "C" fluxbin_status_t fluxbin_plan_create_gated(int32_t n, const fluxbin_weight_t *const *w,
                                                      const uint16_t *const *d_x, const int64_t *ldx,
                                                      void *const *d_y, const int64_t *ldy,
                                                      const int32_t *gate_up, int32_t n_gated,
                                                      int32_t B, int32_t y_is_fp32,
                                                      void *d_table, size_t table_bytes,
                                                      void *d_workspace, size_t ws_bytes,
                                                      void *cuda_stream, fluxbin_plan_t **out)
{
    return plan_create_impl(n, w, d_x, ldx, d_y, ldy, gate_up, n_gated, B, y_is_fp32, d_table, table_bytes, d_workspace, ws_bytes,
                            cuda_stream, out);
}

extern "C" fluxbin_status_t fluxbin_plan_run(const fluxbin_plan_t *plan, void *cuda_stream)
{
    if (!plan) return FLUXBIN_ERR_NULL;
    int dev = -1;
    FB_CUDA(cudaGetDevice(&dev));
    if (dev != plan->device) return FLUXBIN_ERR_UNSUPPORTED;      // the plan's layers live on another device
    cudaStream_t s = (cudaStream_t)cuda_stream;
    fbk::LaunchParams p;
    std::memset(&p.single, 0, sizeof(p.single));
    p.n = plan->n;
    p.y_fp32 = plan->y_fp32;
    p.counters = plan->d_counters;
    for (const PlanChunk &pc : plan->chunks) {
        p.table = pc.d_entries;
        p.cuts = pc.d_cuts;
        p.nb = pc.nb;
        p.nshares = pc.shape.nshares;
        cudaError_t e = launch_kernel(pc.mode, plan->sps0, plan->sps1, pc.shape, p, s);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    return FLUXBIN_OK;
}

extern "C" int32_t fluxbin_plan_num_launches(const fluxbin_plan_t *plan) { return plan ? (int32_t)plan->chunks.size() : -1; }

extern "C" int32_t fluxbin_plan_pairs_per_row_block(const fluxbin_plan_t *plan)
{
    if (!plan || plan->chunks.empty()) return -1;
    return plan->chunks[0].shape.np;       // the plan's first launch
}

extern "C" void fluxbin_plan_free(fluxbin_plan_t *plan) { delete plan; }

extern "C" fluxbin_status_t fluxbin_debug_tables(const fluxbin_weight_t *w, const uint16_t *d_x, int32_t pair,
                                                 float *d_tables, int32_t *h_cols, uint16_t *h_alpha, void *cuda_stream)
{
    if (!w || !d_x || !d_tables) return FLUXBIN_ERR_NULL;
    const int np = w->h.npairs[0] + w->h.npairs[1];
    if (pair < 0 || pair >= np) return FLUXBIN_ERR_RANGE;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    const uint8_t *desc = (const uint8_t *)w->d_packed + w->h.off_coldesc + (size_t)pair * FB_PAIR_DESC_BYTES;
    fbk::fluxbin_debug_tables_kernel<<<1, fbk::Cfg<1>::kThreads, fbk::smem_bytes<1>(), s>>>(desc, d_x, d_tables);
    FB_CUDA(cudaGetLastError());
    if (h_cols || h_alpha) {
        uint16_t tmp[512];
        FB_CUDA(cudaMemcpyAsync(tmp, desc, sizeof(tmp), cudaMemcpyDeviceToHost, s));
        FB_CUDA(cudaStreamSynchronize(s));
        for (int i = 0; i < 256; ++i) {
            if (h_cols) h_cols[i] = tmp[2 * i];
            if (h_alpha) h_alpha[i] = tmp[2 * i + 1];
        }
    }
    return FLUXBIN_OK;
}

#ifdef FB_TRACE
// Instrumented build only: copy the per-CTA phase timestamps of the last launch to the host.
extern "C" int fluxbin_debug_trace(unsigned long long *h_out)
{
    return (int)cudaMemcpyFromSymbol(h_out, fbk::g_fb_trace, sizeof(unsigned long long) * 8 * 1024 * 12);
}
#endif
