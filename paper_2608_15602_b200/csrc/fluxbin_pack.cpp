// Host side of the FluxBin library: validation, the private packed layout, pack / unpack.
// Stage S0 of the path (offline): the canonical bases, scales and salient map (Sec. 3.2,
// Def. 3.5 / Eq. 12-13) are re-tiled into the item stream the lookup kernel consumes.
#include "fluxbin_internal.h"

#include <algorithm>
#include <cstring>
#include <vector>

namespace fb {

static inline int gcd_int(int a, int b) { while (b) { int t = a % b; a = b; b = t; } return a; }

fluxbin_status_t validate_dims(const fluxbin_layer_desc_t *d)
{
    if (!d) return FLUXBIN_ERR_NULL;
    if (d->M < 1 || d->N < 32 || d->N % 32 != 0 || d->N > 65536) return FLUXBIN_ERR_SHAPE;
    if (d->g < 32 || d->g % 32 != 0 || d->N % d->g != 0) return FLUXBIN_ERR_SHAPE;
    if (d->Kb < 1 || d->Kb > 4 || d->Ks < 0 || d->Ks > 4) return FLUXBIN_ERR_RANGE;
    if (d->n_sal < 0 || d->n_sal > d->N) return FLUXBIN_ERR_RANGE;
    if ((int64_t)d->M > (int64_t)1 << 24) return FLUXBIN_ERR_SHAPE;
    return FLUXBIN_OK;
}

static fluxbin_status_t validate_salient(const fluxbin_layer_desc_t *d)
{
    if (d->Ks == 0 || d->n_sal == 0) return FLUXBIN_OK;
    if (!d->sal_idx) return FLUXBIN_ERR_NULL;
    int prev = -1;
    for (int v = 0; v < d->n_sal; ++v) {
        int j = d->sal_idx[v];
        if (j <= prev || j >= d->N) return FLUXBIN_ERR_SALIENT_MAP;
        prev = j;
    }
    return FLUXBIN_OK;
}

// The salient sub-vectors of one base: runs of virtual columns that share a row-scale group are
// padded to whole sub-vectors (when every sub-vector carries its own scale), or the virtual
// columns are simply cut into consecutive sub-vectors (when the layer has a single scale group).
void salient_svecs(const fluxbin_layer_desc_t *d, int sps1, std::vector<SalSvec> &out)
{
    out.clear();
    if (d->Ks == 0 || d->n_sal == 0) return;
    if (sps1 == 16) {
        for (int v = 0; v < d->n_sal; v += 8) out.push_back({v, std::min(8, d->n_sal - v), 0});
        return;
    }
    int v0 = 0;
    while (v0 < d->n_sal) {
        int G = d->sal_idx[v0] / d->g, v1 = v0;
        while (v1 < d->n_sal && d->sal_idx[v1] / d->g == G) ++v1;
        for (int c = v0; c < v1; c += 8) out.push_back({c, std::min(8, v1 - c), G});
        v0 = v1;
    }
}

// Salient units carry one scale per row only when the layer has a single row-scale group and the
// global region is in that format too (g a multiple of 128); otherwise one scale per sub-vector.
static int salient_sps(int N, int g) { return (N / g == 1 && g % 128 == 0) ? 16 : 1; }

static int item_bytes_for(int sps) { return FB_ITEM_BITS_BYTES + 32 * 2 * (32 / sps); }

// table slots of pair P (32, or fewer for a narrow last salient pair) and the bytes of one of its items
static int pair_width(const FbHeader &h, int region, int P)
{
    return (region == 1 && h.sps[1] == 1 && P == h.npairs[1] - 1) ? h.sal_last_w : 32;
}
static int pair_item_bytes(const FbHeader &h, int region, int P)
{
    const int w = pair_width(h, region, P);
    return w == 32 ? h.item_bytes[region] : 96 * w;
}

// Fill every header field.  n_svec < 0 selects the upper bound (salient map unknown).
static void make_header(const fluxbin_layer_desc_t *d, int n_svec, int n_dead, FbHeader &h)
{
    std::memset(&h, 0, sizeof(h));
    h.magic = FB_MAGIC;
    h.version = FB_VERSION;
    h.M = d->M; h.N = d->N; h.Kb = d->Kb; h.g = d->g;
    bool sal = d->Ks > 0 && d->n_sal > 0;
    h.Ks = sal ? d->Ks : 0;
    h.n_sal = sal ? d->n_sal : 0;
    h.Mpad = (d->M + 31) / 32 * 32;
    h.nrb = h.Mpad / 32;
    int ng = d->N / d->g;
    h.sps[0] = gcd_int(d->g, 128) / 8;
    h.sps[1] = salient_sps(d->N, d->g);
    h.sal_last_w = 32;
    int nblk = (d->N + 127) / 128;
    h.nunits[0] = nblk * d->Kb;
    h.npairs[0] = (h.nunits[0] + 1) / 2;
    if (sal) {
        if (n_svec < 0) {
            int runs = std::min(ng, d->n_sal);
            n_svec = (h.sps[1] == 16) ? (d->n_sal + 7) / 8 : (d->n_sal + 7 * runs) / 8;
            n_dead = ng;
        }
        h.n_sal_svec = n_svec;
        h.n_dead = n_dead;
        if (h.sps[1] == 16) {
            // one scale per (row, unit): every base's sub-vectors are padded to whole units of 16
            h.nunits[1] = ((n_svec + 15) / 16) * h.Ks;
            h.npairs[1] = (h.nunits[1] + 1) / 2;
        } else {
            // one scale per (row, sub-vector): the sub-vectors of all bases form one flat list of table slots
            const int slots = n_svec * h.Ks;
            h.nunits[1] = (slots + 15) / 16;
            h.npairs[1] = (slots + 31) / 32;
            const int last = slots - 32 * (h.npairs[1] - 1);
            h.sal_last_w = last <= 8 ? 8 : last <= 16 ? 16 : 32;
        }
    }
    h.item_bytes[0] = item_bytes_for(h.sps[0]);
    h.item_bytes[1] = item_bytes_for(h.sps[1]);
    uint64_t off = FB_HEADER_BYTES;
    h.off_coldesc = off;
    off += (uint64_t)(h.npairs[0] + h.npairs[1]) * FB_PAIR_DESC_BYTES;
    h.off_items[0] = off;
    off += (uint64_t)h.npairs[0] * h.nrb * h.item_bytes[0];
    h.off_items[1] = off;
    if (h.npairs[1] > 0)
        off += (uint64_t)(h.npairs[1] - 1) * h.nrb * h.item_bytes[1] + (uint64_t)h.nrb * pair_item_bytes(h, 1, h.npairs[1] - 1);
    h.off_sal_idx = off;
    off += ((uint64_t)h.n_sal * 4 + 15) / 16 * 16;
    h.off_dead_ids = off;
    off += ((uint64_t)h.n_dead * 4 + 15) / 16 * 16;
    h.off_dead_scales = off;
    off += ((uint64_t)h.Ks * h.n_dead * h.M * 2 + 15) / 16 * 16;
    h.total_bytes = (off + 255) / 256 * 256;
}

static void dead_groups(const fluxbin_layer_desc_t *d, std::vector<int> &dead)
{
    dead.clear();
    if (d->Ks == 0 || d->n_sal == 0) return;
    int ng = d->N / d->g;
    std::vector<char> alive(ng, 0);
    for (int v = 0; v < d->n_sal; ++v) alive[d->sal_idx[v] / d->g] = 1;
    for (int G = 0; G < ng; ++G)
        if (!alive[G]) dead.push_back(G);
}

fluxbin_status_t check_header(const void *p, size_t bytes, FbHeader &h)
{
    if (!p) return FLUXBIN_ERR_NULL;
    if (bytes < FB_HEADER_BYTES) return FLUXBIN_ERR_BUFFER_TOO_SMALL;
    std::memcpy(&h, p, sizeof(h));
    if (h.magic != FB_MAGIC || h.version != FB_VERSION) return FLUXBIN_ERR_FORMAT;
    fluxbin_layer_desc_t d{};
    d.M = h.M; d.N = h.N; d.Kb = h.Kb; d.Ks = h.Ks; d.g = h.g; d.n_sal = h.n_sal;
    if (validate_dims(&d) != FLUXBIN_OK) return FLUXBIN_ERR_FORMAT;
    FbHeader ref;
    make_header(&d, h.n_sal_svec, h.n_dead, ref);
    if (std::memcmp(&ref, &h, sizeof(h)) != 0) return FLUXBIN_ERR_FORMAT;
    return FLUXBIN_OK;
}

fluxbin_status_t validate_dims_and_map(const fluxbin_layer_desc_t *d)
{
    fluxbin_status_t s = validate_dims(d);
    if (s != FLUXBIN_OK) return s;
    return validate_salient(d);
}

void make_packed_header(const fluxbin_layer_desc_t *d, FbHeader &h, std::vector<SalSvec> &sv, std::vector<int> &dead)
{
    salient_svecs(d, salient_sps(d->N, d->g), sv);
    dead_groups(d, dead);
    make_header(d, (int)sv.size(), (int)dead.size(), h);
}

// ---- what a table slot holds: which canonical bits / scales / columns it covers ------------------

struct SlotSrc {
    bool valid = false;
    bool salient = false;
    int k = 0;          // base
    int sv = 0;         // global: sub-vector index (8 columns from sv * 8);  salient: index into the sub-vector list
};

// table slot sigma (0..31) of pair P of a region; n_sv = salient sub-vectors per base
static SlotSrc slot_src(const FbHeader &h, int region, int P, int sigma)
{
    SlotSrc s;
    if (region == 0) {
        const int u = 2 * P + (sigma >> 4);
        if (u >= h.nunits[0]) return s;
        s.valid = true;
        s.k = u % h.Kb;
        s.sv = (u / h.Kb) * 16 + (sigma & 15);
        if (s.sv * 8 >= h.N) s.valid = false;
        return s;
    }
    s.salient = true;
    if (h.sps[1] == 16) {
        const int u = 2 * P + (sigma >> 4), upb = h.nunits[1] / h.Ks;
        if (u >= h.nunits[1]) return s;
        s.k = u / upb;
        s.sv = (u % upb) * 16 + (sigma & 15);
        s.valid = s.sv < h.n_sal_svec;
        return s;
    }
    const int flat = 32 * P + (sigma & (pair_width(h, 1, P) - 1));       // a narrow pair repeats its live tables
    if (flat >= h.n_sal_svec * h.Ks) return s;
    s.valid = true;
    s.k = flat / h.n_sal_svec;
    s.sv = flat % h.n_sal_svec;
    return s;
}

// w (<= 8) bits of a packed row starting at bit position `bit`.
static inline unsigned extract_bits(const uint32_t *row, int bit, int w)
{
    uint64_t lo = row[bit >> 5];
    uint64_t hi = ((bit & 31) + w > 32) ? row[(bit >> 5) + 1] : 0;
    return (unsigned)(((lo | (hi << 32)) >> (bit & 31)) & ((1u << w) - 1u));
}

// out byte c = in byte c ^ m for the 16 bytes held in (lo, hi), little-endian.
static inline void xor_permute16(uint64_t &lo, uint64_t &hi, int m)
{
    if (m & 8) { uint64_t t = lo; lo = hi; hi = t; }
    if (m & 4) { lo = (lo << 32) | (lo >> 32); hi = (hi << 32) | (hi >> 32); }
    if (m & 2) {
        lo = ((lo & 0x0000ffff0000ffffull) << 16) | ((lo >> 16) & 0x0000ffff0000ffffull);
        hi = ((hi & 0x0000ffff0000ffffull) << 16) | ((hi >> 16) & 0x0000ffff0000ffffull);
    }
    if (m & 1) {
        lo = ((lo & 0x00ff00ff00ff00ffull) << 8) | ((lo >> 8) & 0x00ff00ff00ff00ffull);
        hi = ((hi & 0x00ff00ff00ff00ffull) << 8) | ((hi >> 8) & 0x00ff00ff00ff00ffull);
    }
}

static inline void deposit_bits(uint32_t *row, int bit, int w, unsigned val)
{
    for (int n = 0; n < w; ++n)
        if ((val >> n) & 1u) row[(bit + n) >> 5] |= 1u << ((bit + n) & 31);
}

} // namespace fb

using namespace fb;

extern "C" fluxbin_status_t fluxbin_validate(const fluxbin_layer_desc_t *d)
{
    fluxbin_status_t s = validate_dims(d);
    if (s != FLUXBIN_OK) return s;
    if (!d->bits || !d->row_scale || !d->col_scale) return FLUXBIN_ERR_NULL;
    if (d->Ks > 0 && d->n_sal > 0 && (!d->sal_bits || !d->sal_row_scale || !d->sal_col_scale || !d->sal_idx))
        return FLUXBIN_ERR_NULL;
    return validate_salient(d);
}

extern "C" size_t fluxbin_packed_size(const fluxbin_layer_desc_t *d)
{
    if (validate_dims(d) != FLUXBIN_OK) return 0;
    FbHeader h;
    if (d->Ks > 0 && d->n_sal > 0 && d->sal_idx) {
        if (validate_salient(d) != FLUXBIN_OK) return 0;
        int sps1 = salient_sps(d->N, d->g);
        std::vector<SalSvec> sv;
        std::vector<int> dead;
        salient_svecs(d, sps1, sv);
        dead_groups(d, dead);
        make_header(d, (int)sv.size(), (int)dead.size(), h);
    } else {
        make_header(d, -1, 0, h);
    }
    return (size_t)h.total_bytes;
}

extern "C" fluxbin_status_t fluxbin_packed_dims(const void *p, size_t bytes, fluxbin_layer_desc_t *out)
{
    if (!out) return FLUXBIN_ERR_NULL;
    FbHeader h;
    fluxbin_status_t s = check_header(p, bytes, h);
    if (s != FLUXBIN_OK) return s;
    out->M = h.M; out->N = h.N; out->Kb = h.Kb; out->Ks = h.Ks; out->g = h.g; out->n_sal = h.n_sal;
    return FLUXBIN_OK;
}

extern "C" fluxbin_status_t fluxbin_pack_host(const fluxbin_layer_desc_t *d, void *h_packed, size_t bytes)
{
    fluxbin_status_t st = fluxbin_validate(d);
    if (st != FLUXBIN_OK) return st;
    if (!h_packed) return FLUXBIN_ERR_NULL;

    const int sps1 = salient_sps(d->N, d->g);
    std::vector<SalSvec> sv;
    std::vector<int> dead;
    salient_svecs(d, sps1, sv);
    dead_groups(d, dead);
    FbHeader h;
    make_header(d, (int)sv.size(), (int)dead.size(), h);
    if (bytes < h.total_bytes) return FLUXBIN_ERR_BUFFER_TOO_SMALL;

    uint8_t *base = (uint8_t *)h_packed;
    std::memcpy(base, &h, sizeof(h));
    const int M = h.M, N = h.N, Kb = h.Kb, Ks = h.Ks, g = h.g, n_sal = h.n_sal;
    const int ng = N / g, nw = N / 32, nws = (n_sal + 31) / 32;

    // ---- fused column-scale / column-index table (Eq. 11, Eq. 13): one entry per table column
    uint16_t *cd = (uint16_t *)(base + h.off_coldesc);
    for (int region = 0; region < 2; ++region)
        for (int P = 0; P < h.npairs[region]; ++P) {
            uint16_t *pd = cd + (size_t)((region ? h.npairs[0] : 0) + P) * (FB_PAIR_DESC_BYTES / 2);
            for (int sigma = 0; sigma < 32; ++sigma) {
                const SlotSrc ss = slot_src(h, region, P, sigma);
                for (int n = 0; n < 8; ++n) {
                    uint16_t xi = 0, al = 0;
                    if (ss.valid && !ss.salient) {
                        int col = ss.sv * 8 + n;
                        if (col < N) { xi = (uint16_t)col; al = d->col_scale[(size_t)ss.k * N + col]; }
                    } else if (ss.valid && n < sv[ss.sv].w) {
                        int v = sv[ss.sv].vstart + n;
                        xi = (uint16_t)d->sal_idx[v];
                        al = d->sal_col_scale[(size_t)ss.k * n_sal + v];
                    }
                    pd[(sigma * 8 + n) * 2 + 0] = xi;
                    pd[(sigma * 8 + n) * 2 + 1] = al;
                }
            }
        }

    // ---- items: weight bytes in lane-rotated order + row scales in step order
    for (int region = 0; region < 2; ++region) {
        const int sps = h.sps[region];
        const int64_t nitems = (int64_t)h.npairs[region] * h.nrb;
#pragma omp parallel for schedule(static)
        for (int64_t it = 0; it < nitems; ++it) {
            const int P = (int)(it / h.nrb), rb = (int)(it % h.nrb);
            const int w = pair_width(h, region, P), nseg = w / sps;
            uint8_t *item = base + h.off_items[region] + (uint64_t)P * h.nrb * h.item_bytes[region] + (uint64_t)rb * pair_item_bytes(h, region, P);
            uint16_t *sc = (uint16_t *)(item + 32 * w);
            SlotSrc ss[32];
            for (int sigma = 0; sigma < 32; ++sigma) ss[sigma] = slot_src(h, region, P, sigma);
            for (int l = 0; l < 32; ++l) {
                const int row = rb * 32 + l;
                const bool live = row < M;
                // table index and row scale of this row for every table slot of the pair
                alignas(16) uint8_t src[32];
                uint16_t slotscale[32];
                std::memset(src, 0, sizeof(src));
                std::memset(slotscale, 0, sizeof(slotscale));
                if (live && region == 0) {
                    for (int u = 0; u < 2; ++u) {
                        if (!ss[16 * u].valid) continue;
                        const int k = ss[16 * u].k, colb = ss[16 * u].sv * 8;
                        const int nbytes = std::min(16, (N - colb) / 8);   // N % 32 == 0
                        const uint8_t *r = (const uint8_t *)(d->bits + ((size_t)k * M + row) * nw);
                        std::memcpy(src + 16 * u, r + colb / 8, nbytes);   // little-endian words: byte = 8 columns
                        const uint16_t *rs = d->row_scale + ((size_t)k * M + row) * ng;
                        for (int t = 0; t < nbytes; t += sps) slotscale[16 * u + t] = rs[(colb + t * 8) / g];
                    }
                } else if (live) {
                    for (int sigma = 0; sigma < w; ++sigma) {
                        if (!ss[sigma].valid) continue;
                        const SalSvec &q = sv[ss[sigma].sv];
                        const uint32_t *r = d->sal_bits + ((size_t)ss[sigma].k * M + row) * nws;
                        src[sigma] = (uint8_t)extract_bits(r, q.vstart, q.w);
                        slotscale[sigma] = d->sal_row_scale[((size_t)ss[sigma].k * M + row) * ng + q.G];
                    }
                }
                if (w == 32) {
                    // lane l reads slot l ^ s at step s: unit u sits in half u ^ (l >> 4), and inside the
                    // half the byte of sub-vector t sits at position t ^ (l & 15)
                    for (int u = 0; u < 2; ++u) {
                        uint64_t lo, hi;
                        std::memcpy(&lo, src + 16 * u, 8);
                        std::memcpy(&hi, src + 16 * u + 8, 8);
                        xor_permute16(lo, hi, l & 15);
                        uint8_t *dst = item + (u ^ (l >> 4)) * 512 + l * 16;
                        std::memcpy(dst, &lo, 8);
                        std::memcpy(dst + 8, &hi, 8);
                    }
                } else {
                    // narrow item: w steps, the byte of step s is that of live slot (l ^ s) mod w
                    for (int c = 0; c < w; ++c) item[l * w + c] = src[(l ^ c) & (w - 1)];
                }
                for (int j = 0; j < nseg; ++j) {
                    // the segment is the aligned block of sps sub-vectors around slot l ^ (j*sps); its
                    // scale is that of the block's first sub-vector (live sub-vectors form a prefix)
                    const int sigma = (l ^ (j * sps)) & (w - 1);
                    const uint16_t v = slotscale[sigma / sps * sps];
                    if (nseg <= 8) sc[l * nseg + j] = v;
                    else sc[(j >> 3) * 256 + l * 8 + (j & 7)] = v;
                }
            }
        }
    }

    // ---- side data for the exact inverse: salient map and the row scales no virtual column uses
    if (n_sal > 0) std::memcpy(base + h.off_sal_idx, d->sal_idx, (size_t)n_sal * 4);
    if (!dead.empty()) {
        std::memcpy(base + h.off_dead_ids, dead.data(), dead.size() * 4);
        uint16_t *ds = (uint16_t *)(base + h.off_dead_scales);
        for (int k = 0; k < Ks; ++k)
            for (size_t q = 0; q < dead.size(); ++q)
                for (int i = 0; i < M; ++i)
                    ds[((size_t)k * dead.size() + q) * M + i] = d->sal_row_scale[((size_t)k * M + i) * ng + dead[q]];
    }
    // padding bytes between sections stay whatever the caller's buffer held; zero the tail pads
    // that fluxbin_unpack_host never reads so that equal layers give equal buffers
    auto zero_pad = [&](uint64_t from, uint64_t to) { if (to > from) std::memset(base + from, 0, to - from); };
    zero_pad(h.off_sal_idx + (uint64_t)n_sal * 4, h.off_dead_ids);
    zero_pad(h.off_dead_ids + (uint64_t)dead.size() * 4, h.off_dead_scales);
    zero_pad(h.off_dead_scales + (uint64_t)Ks * dead.size() * M * 2, h.total_bytes);
    return FLUXBIN_OK;
}

extern "C" fluxbin_status_t fluxbin_unpack_host(const void *h_packed, size_t bytes, fluxbin_layer_desc_t *out)
{
    if (!out) return FLUXBIN_ERR_NULL;
    FbHeader h;
    fluxbin_status_t st = check_header(h_packed, bytes, h);
    if (st != FLUXBIN_OK) return st;
    if (bytes < h.total_bytes) return FLUXBIN_ERR_BUFFER_TOO_SMALL;
    const uint8_t *base = (const uint8_t *)h_packed;
    const int M = h.M, N = h.N, Kb = h.Kb, Ks = h.Ks, g = h.g, n_sal = h.n_sal;
    const int ng = N / g, nw = N / 32, nws = (n_sal + 31) / 32;
    out->M = M; out->N = N; out->Kb = Kb; out->Ks = Ks; out->g = g; out->n_sal = n_sal;

    uint32_t *bits = (uint32_t *)out->bits;
    uint16_t *row_scale = (uint16_t *)out->row_scale, *col_scale = (uint16_t *)out->col_scale;
    int32_t *sal_idx = (int32_t *)out->sal_idx;
    uint32_t *sal_bits = (uint32_t *)out->sal_bits;
    uint16_t *sal_row_scale = (uint16_t *)out->sal_row_scale, *sal_col_scale = (uint16_t *)out->sal_col_scale;

    if (sal_idx && n_sal > 0) std::memcpy(sal_idx, base + h.off_sal_idx, (size_t)n_sal * 4);
    if (sal_bits) std::memset(sal_bits, 0, (size_t)Ks * M * nws * 4);

    // the salient sub-vector structure is a function of the stored salient map
    fluxbin_layer_desc_t d{};
    d.M = M; d.N = N; d.Kb = Kb; d.Ks = Ks; d.g = g; d.n_sal = n_sal;
    d.sal_idx = (const int32_t *)(base + h.off_sal_idx);
    std::vector<SalSvec> sv;
    salient_svecs(&d, h.sps[1], sv);
    if ((int)sv.size() != h.n_sal_svec) return FLUXBIN_ERR_FORMAT;

    const uint16_t *cd = (const uint16_t *)(base + h.off_coldesc);
    for (int region = 0; region < 2; ++region)
        for (int P = 0; P < h.npairs[region]; ++P) {
            const uint16_t *pd = cd + (size_t)((region ? h.npairs[0] : 0) + P) * (FB_PAIR_DESC_BYTES / 2);
            for (int sigma = 0; sigma < pair_width(h, region, P); ++sigma) {
                const SlotSrc ss = slot_src(h, region, P, sigma);
                if (!ss.valid) continue;
                for (int n = 0; n < 8; ++n) {
                    uint16_t al = pd[(sigma * 8 + n) * 2 + 1];
                    if (!ss.salient) {
                        int col = ss.sv * 8 + n;
                        if (col < N && col_scale) col_scale[(size_t)ss.k * N + col] = al;
                    } else if (n < sv[ss.sv].w && sal_col_scale) {
                        sal_col_scale[(size_t)ss.k * n_sal + sv[ss.sv].vstart + n] = al;
                    }
                }
            }
        }

    for (int region = 0; region < 2; ++region) {
        const int sps = h.sps[region];
        // rows of different items never overlap for global bits/scales; salient bits of one row are
        // touched by several pairs, so the salient region is processed pair-serially per row block
#pragma omp parallel for schedule(static)
        for (int rb = 0; rb < h.nrb; ++rb)
            for (int P = 0; P < h.npairs[region]; ++P) {
                const int w = pair_width(h, region, P), nseg = w / sps;
                const uint8_t *item = base + h.off_items[region] + (uint64_t)P * h.nrb * h.item_bytes[region] + (uint64_t)rb * pair_item_bytes(h, region, P);
                const uint16_t *sc = (const uint16_t *)(item + 32 * w);
                SlotSrc ss[32];
                for (int sigma = 0; sigma < 32; ++sigma) ss[sigma] = slot_src(h, region, P, sigma);
                for (int l = 0; l < 32; ++l) {
                    const int row = rb * 32 + l;
                    if (row >= M) continue;
                    uint8_t src[32];
                    uint16_t slotscale[32];
                    for (int c = 0; c < w; ++c) {
                        const int sigma = (l ^ c) & (w - 1);
                        src[sigma] = (w == 32) ? item[(c >> 4) * 512 + l * 16 + (c & 15)] : item[l * w + c];
                    }
                    for (int j = 0; j < nseg; ++j) {
                        const int sigma0 = (l ^ (j * sps)) & (w - 1);
                        const uint16_t v = (nseg <= 8) ? sc[l * nseg + j] : sc[(j >> 3) * 256 + l * 8 + (j & 7)];
                        for (int q = 0; q < sps; ++q) slotscale[sigma0 ^ q] = v;      // the segment's sub-vectors: an aligned block of sps
                    }
                    for (int sigma = 0; sigma < w; ++sigma) {
                        if (!ss[sigma].valid) continue;
                        const int k = ss[sigma].k;
                        if (!ss[sigma].salient) {
                            const int col0 = ss[sigma].sv * 8;
                            if (bits) {
                                uint8_t *r = (uint8_t *)(bits + ((size_t)k * M + row) * nw);
                                r[col0 >> 3] = src[sigma];     // little-endian words: byte col0/8
                            }
                            if (row_scale && col0 % g == 0) row_scale[((size_t)k * M + row) * ng + col0 / g] = slotscale[sigma];
                        } else {
                            const SalSvec &q = sv[ss[sigma].sv];
                            if (sal_bits) deposit_bits(sal_bits + ((size_t)k * M + row) * nws, q.vstart, q.w, src[sigma]);
                            if (sal_row_scale) sal_row_scale[((size_t)k * M + row) * ng + q.G] = slotscale[sigma];
                        }
                    }
                }
            }
    }

    if (sal_row_scale && h.n_dead > 0) {
        const int32_t *ids = (const int32_t *)(base + h.off_dead_ids);
        const uint16_t *ds = (const uint16_t *)(base + h.off_dead_scales);
        for (int k = 0; k < Ks; ++k)
            for (int q = 0; q < h.n_dead; ++q)
                for (int i = 0; i < M; ++i)
                    sal_row_scale[((size_t)k * M + i) * ng + ids[q]] = ds[((size_t)k * h.n_dead + q) * M + i];
    }
    return FLUXBIN_OK;
}
