// C-ABI entry points that touch the GPU: pack-to-device, attach, unpack-from-device, workspace,
// fluxbin_linear (launch only: no allocation, no synchronisation) and the table test hook.
#include "fluxbin_internal.h"
#include "fluxbin_kernel.cuh"

#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>

using namespace fb;

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
constexpr int kMaxDevices = 64;
DeviceInfo g_dev[kMaxDevices];
std::mutex g_dev_mutex;

template <int S0, int S1, int BT> cudaError_t opt_in()
{
    cudaError_t e = cudaFuncSetAttribute(fbk::fluxbin_linear_kernel<S0, S1, BT, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)fbk::smem_bytes<BT>());
    if (e != cudaSuccess) return e;
    if constexpr (fbk::geom(BT) == 1)
        e = cudaFuncSetAttribute(fbk::fluxbin_linear_kernel<S0, S1, BT, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)fbk::smem_bytes<BT>());
    return e;
}
template <int BT> cudaError_t opt_in_bt()
{
    cudaError_t e;
    if ((e = opt_in<16, 16, BT>()) != cudaSuccess) return e;
    if ((e = opt_in<16, 1, BT>()) != cudaSuccess) return e;
    if ((e = opt_in<8, 1, BT>()) != cudaSuccess) return e;
    if ((e = opt_in<4, 1, BT>()) != cudaSuccess) return e;
    return cudaSuccess;
}

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
            FB_CUDA(opt_in_bt<1>());
            FB_CUDA(opt_in_bt<2>());
            FB_CUDA(opt_in_bt<4>());
            FB_CUDA(opt_in_bt<16 + 2>());
            FB_CUDA(opt_in_bt<16 + 4>());
            FB_CUDA(opt_in_bt<16 + 8>());
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

extern "C" void fluxbin_free(fluxbin_weight_t *w) { delete w; }

extern "C" int32_t fluxbin_num_table_sets(const fluxbin_weight_t *w) { return w ? w->h.npairs[0] + w->h.npairs[1] : -1; }

extern "C" fluxbin_status_t fluxbin_set_table_format(fluxbin_weight_t *w, int32_t format)
{
    if (!w) return FLUXBIN_ERR_NULL;
    if (format != FLUXBIN_TABLES_FP32 && format != FLUXBIN_TABLES_FP16) return FLUXBIN_ERR_RANGE;
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
static int mode_for(int nb, int fmt) { return (fmt == FLUXBIN_TABLES_FP16 && nb >= 2) ? 16 + nvec_for(nb) : nvec_for(nb); }
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

// The two-pairs-per-row-block kernel pays two table builds per run of rows but has the better row loop (one
// reduction per two items, loads requested half an item earlier).  Measured on B200 (batch 1): it wins as soon
// as a CTA's share is worth about 30 plain items (cost 60) -- +11 % with one launch per 70B linear, +15 % with
// one per dependency group, +21 % with one per layer -- and loses below that (4096 x 4096 alone, 18 items per
// CTA: 6.7 -> 7.7 us per call).
#ifndef FB_NP2_MIN
#define FB_NP2_MIN 60
#endif
// How a launch is cut: grid size, the statically dealt part of the cost line, the number of shares, and
// whether the two-pairs-per-row-block kernel runs.
struct LaunchShape {
    long long grid, static_cost;
    int nshares;
    bool couples;
};

template <int S0, int S1, int BT>
static cudaError_t launch_shape(long long total_cost, int num_sms, long long items, long long couple_cost, LaunchShape *out)
{
    static int occ = 0;     // resident CTAs per SM of this instantiation (same on every B200)
    if (occ == 0) {
        int o = 0;
        cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o, fbk::fluxbin_linear_kernel<S0, S1, BT, 1>,
                                                                      fbk::Cfg<BT>::kThreads, fbk::smem_bytes<BT>());
        if (e != cudaSuccess) return e;
        occ = o > 0 ? o : 1;
    }
    long long grid = (long long)num_sms * occ;
    if (items < grid) grid = items;
    // Launches with enough work deal 90 % of it out statically and cut the rest into three small
    // shares per CTA (each worth >= ~200 items), drawn dynamically; small launches stay static.
    constexpr int dyn_pct = 10, dyn_k = 3;
    const long long rest = total_cost * dyn_pct / 100;
    if (dyn_pct > 0 && dyn_k > 0 && rest / (grid * dyn_k) >= 400) {
        out->static_cost = total_cost - rest;
        out->nshares = (int)(grid * (1 + dyn_k));
    } else {
        out->static_cost = total_cost;
        out->nshares = (int)grid;
    }
    out->grid = grid;
    // two pairs per row block when every layer allows it (couple_cost > 0: even pair counts everywhere) and a
    // CTA's share is large enough to pay for the second table build
    out->couples = fbk::geom(BT) == 1 && couple_cost > 0 && out->static_cost / grid >= FB_NP2_MIN;
    return cudaSuccess;
}

template <int S0, int S1, int BT>
static cudaError_t launch(const fbk::LaunchParams &p, int num_sms, long long items, long long couple_cost, cudaStream_t s)
{
    LaunchShape shape;
    cudaError_t se = launch_shape<S0, S1, BT>(p.total_cost, num_sms, items, couple_cost, &shape);
    if (se != cudaSuccess) return se;
    const long long grid = shape.grid;
    const bool couples = shape.couples;
    fbk::LaunchParams q = p;
    q.static_cost = shape.static_cost;
    q.nshares = shape.nshares;
    // launched with programmatic stream serialization: the kernel may start while its predecessor in
    // the stream drains (it waits inside, before touching activations or workspace)
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(fbk::Cfg<BT>::kThreads);
    cfg.dynamicSmemBytes = fbk::smem_bytes<BT>();
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if constexpr (fbk::geom(BT) == 1) {
        if (couples) return cudaLaunchKernelEx(&cfg, fbk::fluxbin_linear_kernel<S0, S1, BT, 2>, q);
    }
    return cudaLaunchKernelEx(&cfg, fbk::fluxbin_linear_kernel<S0, S1, BT, 1>, q);
}

// couple_cost: cost of the largest couple of global pairs over the layers of the launch, or 0 when
// some layer has an odd number of global pairs (then the one-pair kernel runs).
template <int BT> static cudaError_t launch_bt(int s0, int s1, int num_sms, const fbk::LaunchParams &p, long long items,
                                               long long couple_cost, cudaStream_t s)
{
    if (s0 == 16 && s1 == 16) return launch<16, 16, BT>(p, num_sms, items, couple_cost, s);
    if (s0 == 16) return launch<16, 1, BT>(p, num_sms, items, couple_cost, s);
    if (s0 == 8) return launch<8, 1, BT>(p, num_sms, items, couple_cost, s);
    return launch<4, 1, BT>(p, num_sms, items, couple_cost, s);
}

// mode: 1, 2, 4 vectors with fp32 tables, 16 + (2, 4, 8) vectors with fp16 tables; the two-pair kernel exists
// for the modes with 4-byte table entries (1 and 16 + 2; couple_cost is ignored elsewhere)
static cudaError_t launch_mode(int mode, int s0, int s1, int num_sms, const fbk::LaunchParams &p, long long items,
                               long long couple_cost, cudaStream_t s)
{
    switch (mode) {
    case 1: return launch_bt<1>(s0, s1, num_sms, p, items, couple_cost, s);
    case 2: return launch_bt<2>(s0, s1, num_sms, p, items, 0, s);
    case 4: return launch_bt<4>(s0, s1, num_sms, p, items, 0, s);
    case 16 + 2: return launch_bt<16 + 2>(s0, s1, num_sms, p, items, couple_cost, s);
    case 16 + 4: return launch_bt<16 + 4>(s0, s1, num_sms, p, items, 0, s);
    case 16 + 8: return launch_bt<16 + 8>(s0, s1, num_sms, p, items, 0, s);
    }
    return cudaErrorInvalidValue;
}


// Work-split cost model, measured on B200 in units of half a 1152-byte item (about 50 ns per CTA):
// an item with one row scale per sub-vector (3072 bytes) takes about 2x a plain item; building one
// table set (two dependent loads, 8K table entries, two barriers) takes about as long as 22 items
// (re-measured against the current row loop: 28 / 36 / 44 / 56 -> 5.61 / 5.80 / 5.85 / 5.83 TB/s on the stack plan).
constexpr int kBuildCost = 44;
// With four or eight vectors in fp16 table entries an item takes about half the time it takes with fp32 entries,
// a build (more vectors per entry, conversions) does not: measured 44 / 66 / 88 / 132 -> 3.29 / 3.47 / 3.51 / 3.46
// TB/s at batch 4 and 1.73 / 1.81 / 1.81 / 1.81 at batch 8.  (With fp32 entries, batch 2 and 4: no effect.)
#ifndef FB_BCH
#define FB_BCH 88
#endif
static int build_cost_for(int mode)
{
    return (mode == 16 + 4 || mode == 16 + 8) ? FB_BCH : kBuildCost;    // two vectors in fp16 entries: 36 / 44 / 56 / 66 all within 1 %
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

static long long entry_cost(const FbHeader &h, int sps1, int build_cost)
{
    int c[2];
    item_costs(h.sps[0], sps1, c);
    return (long long)h.npairs[0] * (build_cost + (long long)h.nrb * c[0]) +
           (long long)h.npairs[1] * (build_cost + (long long)h.nrb * c[1]) + epilogue_cost(h);
}

static void fill_entry(fbk::LinearEntry &E, const fluxbin_weight_t *w, const uint16_t *x, int64_t ldx, void *y, int64_t ldy,
                       float *acc, unsigned *tickets, long long cost_begin)
{
    E.packed = (const uint8_t *)w->d_packed;
    E.x = x; E.y = y; E.acc = acc; E.tickets = tickets;
    E.ldx = ldx; E.ldy = ldy; E.cost_begin = cost_begin;
    E.off_coldesc = w->h.off_coldesc; E.off_items[0] = w->h.off_items[0]; E.off_items[1] = w->h.off_items[1];
    E.M = w->h.M; E.N = w->h.N; E.Kb = w->h.Kb; E.Mpad = w->h.Mpad; E.nrb = w->h.nrb;
    E.npairs[0] = w->h.npairs[0]; E.npairs[1] = w->h.npairs[1];
    E.tile_rb = w->tile_rb; E.ntiles = w->ntiles; E.reserved = 0;
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
    cudaStream_t s = (cudaStream_t)cuda_stream;

    fbk::LaunchParams p;
    p.table = nullptr;
    p.n = 1;
    p.y_fp32 = y_is_fp32 != 0;
    const int sps1_eff = w->h.npairs[1] > 0 ? w->h.sps[1] : 1;
    item_costs(w->h.sps[0], sps1_eff, p.item_cost);
    const int fmt = w->table_format;
    const int bt_ws = ws_bt(B, fmt);
    float *acc = (float *)d_workspace;
    unsigned *tickets = (unsigned *)((uint8_t *)d_workspace + acc_bytes(w, bt_ws));
    p.counters = (unsigned *)((uint8_t *)d_workspace + acc_bytes(w, bt_ws) + ((size_t)w->ntiles * 4 + 255) / 256 * 256);
    const long long items = (long long)(w->h.npairs[0] + w->h.npairs[1]) * w->h.nrb;

    const size_t ysz = y_is_fp32 ? 4 : 2;
    const Chunks ch = chunks_of(B, fmt, (long long)w->h.total_bytes);
    for (int c = 0; c < ch.n; ++c) {
        const int nb = chunk_nb(ch, fmt, c), b0 = chunk_begin(ch, fmt, c);
        fill_entry(p.single, w, d_x + (int64_t)b0 * ldx, ldx, (uint8_t *)d_y + (size_t)b0 * ldy * ysz, ldy, acc, tickets, 0);
        p.nb = nb;
        const int s1 = w->h.npairs[1] > 0 ? w->h.sps[1] : 1;
        p.build_cost = build_cost_for(mode_for(nb, fmt));
        p.total_cost = entry_cost(w->h, sps1_eff, p.build_cost);
        cudaError_t e = launch_mode(mode_for(nb, fmt), w->h.sps[0], s1, w->num_sms, p, items, couple_cost_of(w->h), s);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    return FLUXBIN_OK;
}

// ---- plans: many layers in one persistent launch -------------------------------------------------

struct fluxbin_plan {
    int n, B, y_fp32, nchunks, table_format;
    int sps0, sps1, num_sms;
    long long items, couple_cost;
    std::vector<int> chunk_nb, chunk_build_cost;     // per chunk: vectors, build cost of its kernel's cost model
    std::vector<long long> chunk_total_cost;
    int item_cost[2];
    const fbk::LinearEntry *d_table;     // [nchunks][n]
    unsigned *d_counters;
};

static size_t entry_ws_bytes(const fluxbin_weight_t *w, int bt)
{
    return acc_bytes(w, bt) + ((size_t)w->ntiles * 4 + 255) / 256 * 256;
}

extern "C" size_t fluxbin_plan_table_bytes(int32_t n, int32_t B)
{
    if (n < 1 || B < 1) return 0;
    // an upper bound over the table formats and the cut of the rest
    const int most = chunks_of(B, FLUXBIN_TABLES_FP32, kSplitRestBytes).n;
    return (size_t)n * sizeof(fbk::LinearEntry) * (size_t)most;
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

extern "C" fluxbin_status_t fluxbin_plan_create(int32_t n, const fluxbin_weight_t *const *w,
                                                const uint16_t *const *d_x, const int64_t *ldx,
                                                void *const *d_y, const int64_t *ldy,
                                                int32_t B, int32_t y_is_fp32,
                                                void *d_table, size_t table_bytes,
                                                void *d_workspace, size_t ws_bytes,
                                                void *cuda_stream, fluxbin_plan_t **out)
{
    if (!out) return FLUXBIN_ERR_NULL;
    *out = nullptr;
    if (!w || !d_x || !ldx || !d_y || !ldy || !d_table || !d_workspace) return FLUXBIN_ERR_NULL;
    if (n < 1 || B < 1) return FLUXBIN_ERR_RANGE;
    if ((((uintptr_t)d_table) & 15) || (((uintptr_t)d_workspace) & 15)) return FLUXBIN_ERR_ALIGNMENT;
    if (table_bytes < fluxbin_plan_table_bytes(n, B)) return FLUXBIN_ERR_BUFFER_TOO_SMALL;
    int sps1 = 0;
    for (int i = 0; i < n; ++i) {
        if (!w[i] || !d_x[i] || !d_y[i]) return FLUXBIN_ERR_NULL;
        if (ldx[i] < w[i]->h.N || ldy[i] < w[i]->h.M) return FLUXBIN_ERR_RANGE;
        if ((((uintptr_t)d_x[i]) & 15) || (((uintptr_t)d_y[i]) & 15)) return FLUXBIN_ERR_ALIGNMENT;
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

    const int fmt = w[0]->table_format;
    long long weight_bytes = 0;
    for (int i = 0; i < n; ++i) weight_bytes += (long long)w[i]->h.total_bytes;
    const Chunks ch = chunks_of(B, fmt, weight_bytes);
    const int nchunks = ch.n, bt = ws_bt(B, fmt);
    const size_t ysz = y_is_fp32 ? 4 : 2;
    fbk::LinearEntry *host = (fbk::LinearEntry *)std::malloc(sizeof(fbk::LinearEntry) * (size_t)n * nchunks);
    if (!host) return FLUXBIN_ERR_UNSUPPORTED;
    fluxbin_plan *p = new (std::nothrow) fluxbin_plan;
    if (!p) { std::free(host); return FLUXBIN_ERR_UNSUPPORTED; }
    long long items = 0;
    for (int c = 0; c < nchunks; ++c) {
        uint8_t *ws = (uint8_t *)d_workspace;
        const int nb = chunk_nb(ch, fmt, c), b0 = chunk_begin(ch, fmt, c);
        const int bc = build_cost_for(mode_for(nb, fmt));
        long long cost = 0;
        items = 0;
        for (int i = 0; i < n; ++i) {
            float *acc = (float *)ws;
            unsigned *tickets = (unsigned *)(ws + acc_bytes(w[i], bt));
            fill_entry(host[(size_t)c * n + i], w[i], d_x[i] + (int64_t)b0 * ldx[i], ldx[i],
                       (uint8_t *)d_y[i] + (size_t)b0 * ldy[i] * ysz, ldy[i], acc, tickets, cost);
            cost += entry_cost(w[i]->h, sps1, bc);
            items += (long long)(w[i]->h.npairs[0] + w[i]->h.npairs[1]) * w[i]->h.nrb;
            ws += entry_ws_bytes(w[i], bt);
        }
        p->chunk_nb.push_back(nb);
        p->chunk_build_cost.push_back(bc);
        p->chunk_total_cost.push_back(cost);
    }
    cudaStream_t s = (cudaStream_t)cuda_stream;
    cudaError_t e = cudaMemcpyAsync(d_table, host, sizeof(fbk::LinearEntry) * (size_t)n * nchunks, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    std::free(host);
    if (e != cudaSuccess) { delete p; return cuda_fail(e); }

    p->n = n; p->B = B; p->y_fp32 = y_is_fp32 != 0; p->nchunks = nchunks; p->table_format = fmt;
    p->sps0 = w[0]->h.sps[0]; p->sps1 = sps1; p->num_sms = w[0]->num_sms;
    p->items = items;
    p->couple_cost = 0;
    {
        bool all_even = true;
        for (int i = 0; i < n; ++i) {
            long long c = couple_cost_of(w[i]->h);
            if (c == 0) all_even = false;
            if (c > p->couple_cost) p->couple_cost = c;
        }
        if (!all_even) p->couple_cost = 0;
    }
    item_costs(p->sps0, sps1, p->item_cost);
    p->d_table = (const fbk::LinearEntry *)d_table;
    p->d_counters = (unsigned *)((uint8_t *)d_workspace + fluxbin_plan_workspace_bytes(n, w, B) - 256);
    *out = p;
    return FLUXBIN_OK;
}

extern "C" fluxbin_status_t fluxbin_plan_run(const fluxbin_plan_t *plan, void *cuda_stream)
{
    if (!plan) return FLUXBIN_ERR_NULL;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    fbk::LaunchParams p;
    std::memset(&p.single, 0, sizeof(p.single));
    p.n = plan->n;
    p.y_fp32 = plan->y_fp32;
    p.item_cost[0] = plan->item_cost[0];
    p.item_cost[1] = plan->item_cost[1];
    p.counters = plan->d_counters;
    for (int c = 0; c < plan->nchunks; ++c) {
        const int nb = plan->chunk_nb[c];
        p.table = plan->d_table + (size_t)c * plan->n;
        p.nb = nb;
        p.build_cost = plan->chunk_build_cost[c];
        p.total_cost = plan->chunk_total_cost[c];
        cudaError_t e = launch_mode(mode_for(nb, plan->table_format), plan->sps0, plan->sps1, plan->num_sms, p, plan->items,
                                    plan->couple_cost, s);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    return FLUXBIN_OK;
}

extern "C" int32_t fluxbin_plan_num_launches(const fluxbin_plan_t *plan) { return plan ? plan->nchunks : -1; }

// the launch shape of a kernel family with 4-byte table entries that reads (sps0, sps1) layers
template <int BT>
static cudaError_t launch_shape_geom1(int s0, int s1, long long total_cost, int num_sms, long long items, long long couple_cost,
                                      LaunchShape *shape)
{
    if (s0 == 16 && s1 == 16) return launch_shape<16, 16, BT>(total_cost, num_sms, items, couple_cost, shape);
    if (s0 == 16) return launch_shape<16, 1, BT>(total_cost, num_sms, items, couple_cost, shape);
    if (s0 == 8) return launch_shape<8, 1, BT>(total_cost, num_sms, items, couple_cost, shape);
    return launch_shape<4, 1, BT>(total_cost, num_sms, items, couple_cost, shape);
}

extern "C" int32_t fluxbin_plan_pairs_per_row_block(const fluxbin_plan_t *plan)
{
    if (!plan) return -1;
    // the two-pair kernel exists for 4-byte table entries only: one vector, or two with fp16 entries
    const int mode = mode_for(plan->chunk_nb[0], plan->table_format);       // the plan's first launch
    LaunchShape shape;
    cudaError_t e;
    if (mode == 1)
        e = launch_shape_geom1<1>(plan->sps0, plan->sps1, plan->chunk_total_cost[0], plan->num_sms, plan->items, plan->couple_cost, &shape);
    else if (mode == 16 + 2)
        e = launch_shape_geom1<16 + 2>(plan->sps0, plan->sps1, plan->chunk_total_cost[0], plan->num_sms, plan->items, plan->couple_cost, &shape);
    else
        return 1;
    if (e != cudaSuccess) return -1;
    return shape.couples ? 2 : 1;
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
    return (int)cudaMemcpyFromSymbol(h_out, fbk::g_fb_trace, sizeof(unsigned long long) * 1024 * 12);
}
#endif
