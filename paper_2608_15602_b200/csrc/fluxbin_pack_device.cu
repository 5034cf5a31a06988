// Stage S0 on the device: fluxbin_pack_device re-tiles canonical arrays that already live in device memory
// (the outputs of fluxbin_rc_decomp and fluxbin_rc_salient_collect) into the packed item stream, byte for byte
// what fluxbin_pack_host writes (Sec. 3.2, Def. 3.5 / Eq. 12-13), so a layer can go from a dense matrix to a
// packed one without its arrays crossing host memory.  Only the salient map is needed on the host: the header and
// the sub-vector structure are functions of it.
//
// fluxbin_rc_salient_collect turns the outputs of the salient refinement (which ran on a padded matrix, one block
// of `width` columns per row-scale group that has salient columns) into the canonical salient arrays.
#include "fluxbin_internal.h"

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <cstring>
#include <vector>

using namespace fb;

#define FB_CUDA(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) return fb::record_cuda_error((int)e_); } while (0)

namespace pkd {

struct Src {                 // canonical arrays, device memory
    const uint32_t *bits;
    const uint16_t *row_scale, *col_scale;
    const int32_t *sal_idx;
    const uint32_t *sal_bits;
    const uint16_t *sal_row_scale, *sal_col_scale;
    const int32_t *svtab;    // [n_sal_svec][3] {first virtual column, live columns, row-scale group}
    const int32_t *dead;     // [n_dead] row-scale groups without salient columns
};

__host__ __device__ inline int pair_width(const FbHeader &h, int region, int P)
{
    return (region == 1 && h.sps[1] == 1 && P == h.npairs[1] - 1) ? h.sal_last_w : 32;
}

// what table slot sigma of pair P holds: returns false for an empty slot; k = base, sv = sub-vector
// (global: 8 columns from sv * 8; salient: index into the sub-vector table)
__device__ inline bool slot_src(const FbHeader &h, int region, int P, int sigma, int &k, int &sv)
{
    if (region == 0) {
        const int u = 2 * P + (sigma >> 4);
        if (u >= h.nunits[0]) return false;
        k = u % h.Kb;
        sv = (u / h.Kb) * 16 + (sigma & 15);
        return sv * 8 < h.N;
    }
    if (h.sps[1] == 16) {
        const int u = 2 * P + (sigma >> 4), upb = h.nunits[1] / h.Ks;
        if (u >= h.nunits[1]) return false;
        k = u / upb;
        sv = (u % upb) * 16 + (sigma & 15);
        return sv < h.n_sal_svec;
    }
    const int flat = 32 * P + (sigma & (pair_width(h, 1, P) - 1));
    if (flat >= h.n_sal_svec * h.Ks) return false;
    k = flat / h.n_sal_svec;
    sv = flat % h.n_sal_svec;
    return true;
}

// w (<= 8) bits of a packed row starting at bit position `bit`
__device__ inline unsigned extract_bits(const uint32_t *row, int bit, int w)
{
    unsigned long long lo = row[bit >> 5];
    unsigned long long hi = ((bit & 31) + w > 32) ? row[(bit >> 5) + 1] : 0ull;
    return (unsigned)(((lo | (hi << 32)) >> (bit & 31)) & ((1u << w) - 1u));
}

// fused column-scale / column-index table: one thread per (pair, slot, n)
__global__ void coldesc_kernel(FbHeader h, Src s, uint16_t *cd)
{
    const long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    const long long total = (long long)(h.npairs[0] + h.npairs[1]) * 256;
    if (i >= total) return;
    const int n = (int)(i & 7), sigma = (int)((i >> 3) & 31), Pg = (int)(i >> 8);
    const int region = Pg >= h.npairs[0], P = region ? Pg - h.npairs[0] : Pg;
    int k = 0, sv = 0;
    uint16_t xi = 0, al = 0;
    if (slot_src(h, region, P, sigma, k, sv)) {
        if (!region) {
            const int col = sv * 8 + n;
            if (col < h.N) { xi = (uint16_t)col; al = s.col_scale[(size_t)k * h.N + col]; }
        } else if (n < s.svtab[3 * sv + 1]) {
            const int v = s.svtab[3 * sv] + n;
            xi = (uint16_t)s.sal_idx[v];
            al = s.sal_col_scale[(size_t)k * h.n_sal + v];
        }
    }
    cd[i * 2] = xi;
    cd[i * 2 + 1] = al;
}

// items: one warp per item, lane = row of the item
__global__ void __launch_bounds__(256) items_kernel(FbHeader h, Src s, uint8_t *base, int region)
{
    const int lane = threadIdx.x & 31;
    const long long it = blockIdx.x * (long long)(blockDim.x >> 5) + (threadIdx.x >> 5);
    if (it >= (long long)h.npairs[region] * h.nrb) return;
    const int P = (int)(it / h.nrb), rb = (int)(it % h.nrb);
    const int sps = h.sps[region], w = pair_width(h, region, P), nseg = w / sps;
    const int ib = w == 32 ? h.item_bytes[region] : 96 * w;
    uint8_t *item = base + h.off_items[region] + (unsigned long long)P * h.nrb * h.item_bytes[region] + (unsigned long long)rb * ib;
    uint16_t *sc = (uint16_t *)(item + 32 * w);
    const int row = rb * 32 + lane, ng = h.N / h.g, nw = h.N / 32, nws = (h.n_sal + 31) / 32;
    const bool live = row < h.M;
    // table index and row scale of this row for every table slot of the pair
    uint8_t src[32];
    uint16_t slotscale[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) { src[i] = 0; slotscale[i] = 0; }
    for (int sigma = 0; sigma < w; ++sigma) {
        int k = 0, sv = 0;
        if (!live || !slot_src(h, region, P, sigma, k, sv)) continue;
        if (!region) {
            src[sigma] = ((const uint8_t *)(s.bits + ((size_t)k * h.M + row) * nw))[sv];      // little-endian words: byte = 8 columns
            slotscale[sigma] = s.row_scale[((size_t)k * h.M + row) * ng + (sv * 8) / h.g];
        } else {
            const int vstart = s.svtab[3 * sv], wv = s.svtab[3 * sv + 1], G = s.svtab[3 * sv + 2];
            src[sigma] = (uint8_t)extract_bits(s.sal_bits + ((size_t)k * h.M + row) * nws, vstart, wv);
            slotscale[sigma] = s.sal_row_scale[((size_t)k * h.M + row) * ng + G];
        }
    }
    // lane l reads slot l ^ s at step s: the byte of step s is that of slot (l ^ s) (mod w for a narrow item)
    for (int c = 0; c < w; ++c) {
        const uint8_t b = src[(lane ^ c) & (w - 1)];
        if (w == 32) item[(c >> 4) * 512 + lane * 16 + (c & 15)] = b;
        else item[lane * w + c] = b;
    }
    for (int j = 0; j < nseg; ++j) {
        // the segment is the aligned block of sps sub-vectors around slot l ^ (j * sps); its scale is that of the
        // block's first sub-vector
        const int sigma = (lane ^ (j * sps)) & (w - 1);
        const uint16_t v = slotscale[sigma / sps * sps];
        if (nseg <= 8) sc[lane * nseg + j] = v;
        else sc[(j >> 3) * 256 + lane * 8 + (j & 7)] = v;
    }
}

// salient row scales of the groups no virtual column uses (kept so that unpacking is an exact inverse)
__global__ void dead_scales_kernel(FbHeader h, Src s, uint16_t *ds)
{
    const long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    const long long total = (long long)h.Ks * h.n_dead * h.M;
    if (i >= total) return;
    const int row = (int)(i % h.M), q = (int)((i / h.M) % h.n_dead), k = (int)(i / ((long long)h.M * h.n_dead));
    ds[i] = s.sal_row_scale[((size_t)k * h.M + row) * (h.N / h.g) + s.dead[q]];
}

// ---- canonical salient arrays from the refinement's outputs on the padded matrix -----------------------------
__global__ void collect_bits_kernel(const uint32_t *bits_p, const int32_t *pos, int Ks, int M, int n_sal, int nwp, uint32_t *out)
{
    const int nws = (n_sal + 31) / 32;
    const long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    if (i >= (long long)Ks * M * nws) return;
    const int wd = (int)(i % nws);
    const long long km = i / nws;                       // k * M + row
    const uint32_t *rowp = bits_p + km * nwp;
    uint32_t word = 0u;
    for (int b = 0; b < 32; ++b) {
        const int v = wd * 32 + b;
        if (v >= n_sal) break;
        const int p = pos[v];
        word |= ((rowp[p >> 5] >> (p & 31)) & 1u) << b;
    }
    out[i] = word;
}
__global__ void collect_row_scales_kernel(const float *rs_p, const int32_t *block_group, int Ks, int M, int nblocks, int ng,
                                          uint16_t *out, float *out_f32)
{
    const long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    if (i >= (long long)Ks * M * nblocks) return;
    const int b = (int)(i % nblocks);
    const long long km = i / nblocks;
    const float v = rs_p[i];
    out[km * ng + block_group[b]] = __half_as_ushort(__float2half_rn(v));
    if (out_f32) out_f32[km * ng + block_group[b]] = v;
}
__global__ void collect_col_scales_kernel(const float *cs_p, const int32_t *pos, int Ks, int n_sal, int ncols_p, uint16_t *out,
                                          float *out_f32)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= Ks * n_sal) return;
    const int k = i / n_sal, v = i % n_sal;
    const float x = cs_p[(size_t)k * ncols_p + pos[v]];
    out[i] = __half_as_ushort(__float2half_rn(x));
    if (out_f32) out_f32[i] = x;
}

} // namespace pkd

static size_t align256(size_t n) { return (n + 255) / 256 * 256; }

extern "C" size_t fluxbin_pack_device_workspace_size(int32_t N, int32_t g, int32_t n_sal)
{
    if (N < 32 || g < 32 || N % g != 0 || n_sal < 0 || n_sal > N) return 0;
    // sub-vector table (at most one sub-vector per salient column) and the list of groups without salient columns
    return align256((size_t)n_sal * 12 + 16) + align256((size_t)(N / g) * 4 + 16);
}

extern "C" fluxbin_status_t fluxbin_pack_device(const fluxbin_layer_desc_t *d_desc, const int32_t *h_sal_idx, void *d_packed,
                                                size_t d_bytes, void *d_workspace, size_t ws_bytes, void *cuda_stream,
                                                fluxbin_weight_t **out)
{
    if (!out || !d_packed || !d_desc || !d_workspace) return FLUXBIN_ERR_NULL;
    *out = nullptr;
    // the descriptor's dimensions and the host copy of the salient map go through the ordinary validation
    fluxbin_layer_desc_t dims = *d_desc;
    const bool sal = dims.Ks > 0 && dims.n_sal > 0;
    if (sal && !h_sal_idx) return FLUXBIN_ERR_NULL;
    dims.sal_idx = h_sal_idx;
    fluxbin_status_t st = validate_dims_and_map(&dims);
    if (st != FLUXBIN_OK) return st;
    if (!d_desc->bits || !d_desc->row_scale || !d_desc->col_scale) return FLUXBIN_ERR_NULL;
    if (sal && (!d_desc->sal_bits || !d_desc->sal_row_scale || !d_desc->sal_col_scale || !d_desc->sal_idx)) return FLUXBIN_ERR_NULL;
    const size_t bytes = fluxbin_packed_size(&dims);
    if (bytes == 0) return FLUXBIN_ERR_SHAPE;
    if (d_bytes < bytes) return FLUXBIN_ERR_BUFFER_TOO_SMALL;
    if (((uintptr_t)d_packed & 15) != 0 || ((uintptr_t)d_workspace & 15) != 0) return FLUXBIN_ERR_ALIGNMENT;
    if (ws_bytes < fluxbin_pack_device_workspace_size(dims.N, dims.g, dims.n_sal)) return FLUXBIN_ERR_BUFFER_TOO_SMALL;

    FbHeader h;
    std::vector<SalSvec> sv;
    std::vector<int> dead;
    make_packed_header(&dims, h, sv, dead);
    std::vector<int32_t> svtab(sv.size() * 3 + 1);
    for (size_t i = 0; i < sv.size(); ++i) { svtab[3 * i] = sv[i].vstart; svtab[3 * i + 1] = sv[i].w; svtab[3 * i + 2] = sv[i].G; }

    cudaStream_t s = (cudaStream_t)cuda_stream;
    uint8_t *base = (uint8_t *)d_packed;
    uint8_t *ws = (uint8_t *)d_workspace;
    int32_t *d_svtab = (int32_t *)ws;
    int32_t *d_dead = (int32_t *)(ws + align256((size_t)dims.n_sal * 12 + 16));
    // everything behind the items starts out zero (the pads between the side sections)
    FB_CUDA(cudaMemsetAsync(base + h.off_sal_idx, 0, (size_t)(h.total_bytes - h.off_sal_idx), s));
    FB_CUDA(cudaMemcpyAsync(base, &h, sizeof(h), cudaMemcpyHostToDevice, s));
    if (!sv.empty()) FB_CUDA(cudaMemcpyAsync(d_svtab, svtab.data(), sv.size() * 12, cudaMemcpyHostToDevice, s));
    if (!dead.empty()) {
        FB_CUDA(cudaMemcpyAsync(d_dead, dead.data(), dead.size() * 4, cudaMemcpyHostToDevice, s));
        FB_CUDA(cudaMemcpyAsync(base + h.off_dead_ids, dead.data(), dead.size() * 4, cudaMemcpyHostToDevice, s));
    }
    if (h.n_sal > 0) FB_CUDA(cudaMemcpyAsync(base + h.off_sal_idx, h_sal_idx, (size_t)h.n_sal * 4, cudaMemcpyHostToDevice, s));

    pkd::Src src;
    src.bits = d_desc->bits; src.row_scale = d_desc->row_scale; src.col_scale = d_desc->col_scale;
    src.sal_idx = d_desc->sal_idx; src.sal_bits = d_desc->sal_bits; src.sal_row_scale = d_desc->sal_row_scale;
    src.sal_col_scale = d_desc->sal_col_scale; src.svtab = d_svtab; src.dead = d_dead;
    const long long ncd = (long long)(h.npairs[0] + h.npairs[1]) * 256;
    pkd::coldesc_kernel<<<(unsigned)((ncd + 255) / 256), 256, 0, s>>>(h, src, (uint16_t *)(base + h.off_coldesc));
    for (int region = 0; region < 2; ++region) {
        const long long nitems = (long long)h.npairs[region] * h.nrb;
        if (nitems > 0) pkd::items_kernel<<<(unsigned)((nitems + 7) / 8), 256, 0, s>>>(h, src, base, region);
    }
    const long long nds = (long long)h.Ks * h.n_dead * h.M;
    if (nds > 0) pkd::dead_scales_kernel<<<(unsigned)((nds + 255) / 256), 256, 0, s>>>(h, src, (uint16_t *)(base + h.off_dead_scales));
    FB_CUDA(cudaGetLastError());
    FB_CUDA(cudaStreamSynchronize(s));          // the host-side tables above are read by the copies until here
    return fluxbin_attach(&h, sizeof(h), d_packed, d_bytes, out);
}

extern "C" fluxbin_status_t fluxbin_rc_salient_collect(const uint32_t *d_bits_p, const float *d_row_scale_p_f32,
                                                       const float *d_col_scale_p_f32, const int32_t *d_pos,
                                                       const int32_t *d_block_group, int32_t M, int32_t N, int32_t g, int32_t Ks,
                                                       int32_t n_sal, int32_t width, int32_t nblocks, uint32_t *d_sal_bits,
                                                       uint16_t *d_sal_row_scale, uint16_t *d_sal_col_scale,
                                                       float *d_sal_row_scale_f32, float *d_sal_col_scale_f32, void *cuda_stream)
{
    if (!d_bits_p || !d_row_scale_p_f32 || !d_col_scale_p_f32 || !d_pos || !d_block_group || !d_sal_bits || !d_sal_row_scale ||
        !d_sal_col_scale)
        return FLUXBIN_ERR_NULL;
    if (M < 1 || N < 32 || g < 32 || N % g != 0 || width < 32 || width % 32 != 0 || nblocks < 1 || nblocks > N / g) return FLUXBIN_ERR_SHAPE;
    if (Ks < 1 || Ks > 4 || n_sal < 1 || n_sal > N || (long long)n_sal > (long long)width * nblocks) return FLUXBIN_ERR_RANGE;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    const int ng = N / g, ncols_p = width * nblocks, nws = (n_sal + 31) / 32;
    FB_CUDA(cudaMemsetAsync(d_sal_row_scale, 0, (size_t)Ks * M * ng * 2, s));
    if (d_sal_row_scale_f32) FB_CUDA(cudaMemsetAsync(d_sal_row_scale_f32, 0, (size_t)Ks * M * ng * 4, s));
    const long long nb = (long long)Ks * M * nws, nr = (long long)Ks * M * nblocks;
    pkd::collect_bits_kernel<<<(unsigned)((nb + 255) / 256), 256, 0, s>>>(d_bits_p, d_pos, Ks, M, n_sal, ncols_p / 32, d_sal_bits);
    pkd::collect_row_scales_kernel<<<(unsigned)((nr + 255) / 256), 256, 0, s>>>(d_row_scale_p_f32, d_block_group, Ks, M, nblocks, ng,
                                                                               d_sal_row_scale, d_sal_row_scale_f32);
    pkd::collect_col_scales_kernel<<<(Ks * n_sal + 255) / 256, 256, 0, s>>>(d_col_scale_p_f32, d_pos, Ks, n_sal, ncols_p,
                                                                            d_sal_col_scale, d_sal_col_scale_f32);
    FB_CUDA(cudaGetLastError());
    return FLUXBIN_OK;
}
