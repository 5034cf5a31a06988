// FluxBin decode linear layer: the LUT GEMV kernel for sm_100a (no tensor cores: the path is a
// table-lookup GEMV bound by HBM and by the shared-memory lookup rate).
//
// One persistent CTA per SM.  The work of a layer is the list of items (pair, row block): a pair
// is one table set (32 tables = two units of 16 sub-vectors), a row block is 32 output rows.
// Items are ordered pair-major and cut into equal contiguous shares, so a CTA builds the tables
// of one or two pairs (stage (i), Eq. 14, column scale fused per Eq. 11) and then streams the
// weight bytes of a long run of rows through them (stage (ii), Eq. 15).  Row scales are applied
// per (row, segment) in registers and the per-row partial sums of this K slice are added to an
// fp32 accumulator in global memory (stage (iii)); the CTA that completes a tile of rows -- found
// with one arrival counter per tile, never by waiting -- converts the tile to the output type and
// re-zeroes the accumulator.
//
// Shared-memory table layout: entry p of table slot sigma lives at shared-window address
// 0x10000 + p*256 + sigma*4*BT  (BT = batch vectors per launch, their entries side by side; for
// BT = 4 the two units of a pair get separate 64 KB planes at 0x10000 and 0x20000).
// A lane at step s reads slot  lane ^ s, so the 32 lanes of a warp always hit 32 different slots:
// every lookup is bank-conflict free by construction, and the packer has stored each lane's
// weight bytes in exactly that order, so the byte of step s sits at a compile-time position.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "fluxbin_layout.h"

namespace fbk {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxTiles = 1024;
constexpr uint32_t kSmallBytes = 256 * 4 * 4 + kMaxTiles * 4;   // scale-fusion scratch + tile counters

struct LinearParams {
    const uint8_t *packed;
    const uint16_t *x;
    int64_t ldx;
    void *y;
    int64_t ldy;
    int y_fp32;
    int nb;              // live batch rows (<= BT)
    float *acc;          // [BT][Mpad] split-K accumulators, zero on entry and on exit
    unsigned *tickets;   // [ntiles] arrival counters, zero on entry and on exit
    int M, Mpad, nrb;
    int npairs[2];
    int item_bytes[2];
    unsigned long long off_coldesc, off_items[2];
    int tile_rb, ntiles;
};

// The tables start at shared-window address 0x10000 so that the address of entry p of a slot is
// (lane constant) | p << 8 with the p byte dropped in by one PRMT and nothing to add.
constexpr uint32_t kTabBase = 0x10000u;

template <int BT> struct TabCfg {
    static constexpr int kTableBytes = (BT == 4) ? 131072 : 65536;
    // address bits of slot sigma at step 0 (table base included); entry p adds p << 8
    __host__ __device__ static constexpr uint32_t lane_const(uint32_t sigma)
    {
        return BT == 1 ? (kTabBase | sigma * 4u)
             : BT == 2 ? (kTabBase | sigma * 8u)
                       : ((kTabBase << (sigma >> 4)) | ((sigma & 15u) * 16u));
    }
    // lane_const(lane ^ s) == lane_const(lane) ^ step_const(s)
    __host__ __device__ static constexpr uint32_t step_const(uint32_t s)
    {
        return BT == 1 ? s * 4u : BT == 2 ? s * 8u : (((s >> 4) ? 0x30000u : 0u) | ((s & 15u) * 16u));
    }
};

__device__ __forceinline__ float h2f(uint32_t bits16) { return __half2float(__ushort_as_half((unsigned short)bits16)); }

__device__ __forceinline__ uint4 ldg_stream_v4(const void *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ uint2 ldg_stream_v2(const void *p)
{
    uint2 v;
    asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
    return v;
}
__device__ __forceinline__ uint32_t ldg_stream_u32(const void *p)
{
    uint32_t v;
    asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
}

template <int BT> struct Vec;
template <> struct Vec<1> { float v[1]; };
template <> struct Vec<2> { float v[2]; };
template <> struct Vec<4> { float v[4]; };

template <int BT> __device__ __forceinline__ Vec<BT> lds_entry(uint32_t addr)
{
    Vec<BT> r;
    if constexpr (BT == 1) asm volatile("ld.shared.f32 %0, [%1];" : "=f"(r.v[0]) : "r"(addr));
    else if constexpr (BT == 2) asm volatile("ld.shared.v2.f32 {%0,%1}, [%2];" : "=f"(r.v[0]), "=f"(r.v[1]) : "r"(addr));
    else asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];"
                      : "=f"(r.v[0]), "=f"(r.v[1]), "=f"(r.v[2]), "=f"(r.v[3]) : "r"(addr));
    return r;
}

template <int BT> __device__ __forceinline__ void sts_entry(uint32_t addr, const float *v)
{
    if constexpr (BT == 1) asm volatile("st.shared.f32 [%0], %1;" ::"r"(addr), "f"(v[0]));
    else if constexpr (BT == 2) asm volatile("st.shared.v2.f32 [%0], {%1,%2};" ::"r"(addr), "f"(v[0]), "f"(v[1]));
    else asm volatile("st.shared.v4.f32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]));
}

// ---------------------------------------------------------------------------------------------
// Stage (i): LUT building with scale fusion (Eq. 14 with a_n = x[col_n] * alpha_c[col_n], Eq. 11;
// for salient tables col_n = sal_idx[v] and alpha = gathered scale, Eq. 13).
// abuf: shared scratch of 32*8*BT floats.  Ends with the tables visible to the whole CTA.
// ---------------------------------------------------------------------------------------------
template <int BT>
__device__ __forceinline__ void build_tables(const uint8_t *pair_desc, const uint16_t *x, int64_t ldx, int nb,
                                             float *abuf)
{
    const int tid = threadIdx.x;
    if (tid < 256) {
        uint32_t e = __ldg((const uint32_t *)pair_desc + tid);   // {u16 column, fp16 alpha} of (slot tid/8, n tid%8)
        uint32_t col = e & 0xffffu;
        float al = h2f(e >> 16);
#pragma unroll
        for (int b = 0; b < BT; ++b) {
            float xv = (b < nb) ? h2f(__ldg(x + (int64_t)b * ldx + col)) : 0.f;
            abuf[tid * BT + b] = xv * al;     // exact in fp32: two 11-bit significands
        }
    }
    __syncthreads();
    const int lane = tid & 31, warp = tid >> 5;
    constexpr int PW = 256 / kWarps;          // table entries per warp: p = warp*PW + q
    constexpr int LOW = (PW == 16) ? 4 : (PW == 32) ? 5 : 3;
    static_assert((1 << LOW) == PW, "warps per CTA must be 8, 16 or 32");
    float a[8][BT];
#pragma unroll
    for (int n = 0; n < 8; ++n)
#pragma unroll
        for (int b = 0; b < BT; ++b) a[n][b] = abuf[(lane * 8 + n) * BT + b];
    float v[PW][BT];
#pragma unroll
    for (int b = 0; b < BT; ++b) {
        float base = 0.f;
#pragma unroll
        for (int n = 7; n >= LOW; --n) base += ((warp * PW) >> n & 1) ? a[n][b] : -a[n][b];
#pragma unroll
        for (int n = LOW - 1; n >= 0; --n) base -= a[n][b];
        v[0][b] = base;
#pragma unroll
        for (int n = 0; n < LOW; ++n)
#pragma unroll
            for (int q = 0; q < (1 << n); ++q) v[q | (1 << n)][b] = v[q][b] + 2.f * a[n][b];
    }
#pragma unroll
    for (int q = 0; q < PW; ++q)
        sts_entry<BT>(TabCfg<BT>::lane_const((uint32_t)lane) | ((uint32_t)(warp * PW + q) << 8), v[q]);
    __syncthreads();
}

// ---------------------------------------------------------------------------------------------
// Stage (ii)+(iii) for one run of row blocks of one pair.
// SPS = sub-vectors per row-scale segment (16: one scale per unit and row; 1: one per sub-vector).
// ---------------------------------------------------------------------------------------------
template <int SPS> struct ItemRegs {
    uint4 b0, b1;                         // weight bytes of steps 0..15 / 16..31
    uint32_t sc[(SPS == 16) ? 1 : (SPS == 8) ? 2 : (SPS == 4) ? 4 : 16];
};

template <int SPS> __device__ __forceinline__ void load_item(ItemRegs<SPS> &r, const uint8_t *item, int lane)
{
    r.b0 = ldg_stream_v4(item + lane * 16);
    r.b1 = ldg_stream_v4(item + 512 + lane * 16);
    const uint8_t *s = item + FB_ITEM_BITS_BYTES;
    if constexpr (SPS == 16) r.sc[0] = ldg_stream_u32(s + lane * 4);
    else if constexpr (SPS == 8) { uint2 t = ldg_stream_v2(s + lane * 8); r.sc[0] = t.x; r.sc[1] = t.y; }
    else if constexpr (SPS == 4) { uint4 t = ldg_stream_v4(s + lane * 16); r.sc[0] = t.x; r.sc[1] = t.y; r.sc[2] = t.z; r.sc[3] = t.w; }
    else {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            uint4 t = ldg_stream_v4(s + q * 512 + lane * 16);
            r.sc[4 * q] = t.x; r.sc[4 * q + 1] = t.y; r.sc[4 * q + 2] = t.z; r.sc[4 * q + 3] = t.w;
        }
    }
}

template <int SPS, int BT>
__device__ __forceinline__ void compute_item(const ItemRegs<SPS> &r, uint32_t tab_lane, float (&out)[BT])
{
    constexpr int NSEG = 32 / SPS;
    const uint32_t w[8] = {r.b0.x, r.b0.y, r.b0.z, r.b0.w, r.b1.x, r.b1.y, r.b1.z, r.b1.w};
#pragma unroll
    for (int b = 0; b < BT; ++b) out[b] = 0.f;
#pragma unroll
    for (int j = 0; j < NSEG; ++j) {
        float s0[BT], s1[BT];
#pragma unroll
        for (int b = 0; b < BT; ++b) { s0[b] = 0.f; s1[b] = 0.f; }
#pragma unroll
        for (int q = 0; q < SPS; ++q) {
            const int s = j * SPS + q;
            // table index byte -> p << 8; the rest of the address is (lane constant) xor (step constant)
            uint32_t idx = __byte_perm(w[s >> 2], 0u, 0x4404u | ((uint32_t)(s & 3) << 4));
            uint32_t addr = idx | (tab_lane ^ TabCfg<BT>::step_const((uint32_t)s));
            Vec<BT> e = lds_entry<BT>(addr);
#pragma unroll
            for (int b = 0; b < BT; ++b) {
                if (q & 1) s1[b] += e.v[b]; else s0[b] += e.v[b];
            }
        }
        float scale = h2f((r.sc[j >> 1] >> ((j & 1) * 16)) & 0xffffu);
#pragma unroll
        for (int b = 0; b < BT; ++b) out[b] = fmaf(scale, s0[b] + s1[b], out[b]);
    }
}

template <int SPS, int BT>
__device__ __forceinline__ void process_rows(const uint8_t *pair_items, int item_bytes, int rb_lo, int rb_hi,
                                             float *acc, int Mpad)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t tab_lane = TabCfg<BT>::lane_const((uint32_t)lane);
    int rb = rb_lo + warp;
    if (rb >= rb_hi) return;
    ItemRegs<SPS> cur, nxt;
    load_item<SPS>(cur, pair_items + (int64_t)rb * item_bytes, lane);
    for (; rb < rb_hi; rb += kWarps) {
        const int rbn = rb + kWarps;
        if (rbn < rb_hi) load_item<SPS>(nxt, pair_items + (int64_t)rbn * item_bytes, lane);
        float out[BT];
        compute_item<SPS, BT>(cur, tab_lane, out);
#pragma unroll
        for (int b = 0; b < BT; ++b) atomicAdd(acc + (int64_t)b * Mpad + rb * 32 + lane, out[b]);
        cur = nxt;
    }
}

template <int SPS0, int SPS1, int BT>
__global__ void __launch_bounds__(kThreads, 1) fluxbin_linear_kernel(const __grid_constant__ LinearParams P)
{
    // dynamic shared memory: [base, 0x10000) holds the small buffers, [0x10000, ...) the tables
    extern __shared__ __align__(16) uint8_t smem[];
    float *abuf = (float *)smem;
    int *tile_cnt = (int *)(abuf + 256 * BT);
    const int tid = threadIdx.x;
    if ((uint32_t)__cvta_generic_to_shared(smem) + kSmallBytes > kTabBase) return;   // host probes this first

    for (int t = tid; t < P.ntiles; t += kThreads) tile_cnt[t] = 0;

    // equal shares of the item list, weighted by item bytes
    const long long I0 = (long long)P.npairs[0] * P.nrb, I1 = (long long)P.npairs[1] * P.nrb;
    const long long w0 = P.item_bytes[0], w1 = P.item_bytes[1];
    const long long T0 = I0 * w0, T = T0 + I1 * w1;
    auto first_item = [&](long long pos) -> long long {
        if (pos <= 0) return 0;
        if (pos >= T) return I0 + I1;
        long long i = (pos + w0 - 1) / w0;
        if (i < I0) return i;
        long long r = pos - T0;
        return I0 + (r <= 0 ? 0 : (r + w1 - 1) / w1);
    };
    long long cur = first_item(T * (long long)blockIdx.x / gridDim.x);
    const long long end = first_item(T * (long long)(blockIdx.x + 1) / gridDim.x);

    while (cur < end) {
        const int region = cur >= I0;
        const long long local = region ? cur - I0 : cur;
        const int pair = (int)(local / P.nrb), rb_lo = (int)(local % P.nrb);
        const long long seg_end = min(end, cur - rb_lo + P.nrb);
        const int rb_hi = rb_lo + (int)(seg_end - cur);

        __syncthreads();     // previous segment's lookups are done before the tables are overwritten
        const uint8_t *desc = P.packed + P.off_coldesc + (size_t)((region ? P.npairs[0] : 0) + pair) * FB_PAIR_DESC_BYTES;
        build_tables<BT>(desc, P.x, P.ldx, P.nb, abuf);
        const uint8_t *items = P.packed + P.off_items[region] + (size_t)pair * P.nrb * P.item_bytes[region];
        if (region == 0) process_rows<SPS0, BT>(items, P.item_bytes[0], rb_lo, rb_hi, P.acc, P.Mpad);
        else process_rows<SPS1, BT>(items, P.item_bytes[1], rb_lo, rb_hi, P.acc, P.Mpad);

        // how many items this CTA contributed to each tile of rows
        const int t_lo = rb_lo / P.tile_rb, t_hi = (rb_hi - 1) / P.tile_rb;
        for (int t = t_lo + tid; t <= t_hi; t += kThreads) {
            int lo = max(rb_lo, t * P.tile_rb), hi = min(rb_hi, (t + 1) * P.tile_rb);
            tile_cnt[t] += hi - lo;          // one thread per tile, segments are serial: no race
        }
        cur = seg_end;
    }

    // Stage (iii): publish, take a ticket per touched tile; the last arrival finishes the tile.
    __threadfence();
    __syncthreads();
    const int npairs = P.npairs[0] + P.npairs[1];
    for (int t = tid; t < P.ntiles; t += kThreads) {
        int c = tile_cnt[t];
        int last = 0;
        if (c > 0) {
            int rbs = min(P.tile_rb, P.nrb - t * P.tile_rb);
            unsigned old = atomicAdd(P.tickets + t, (unsigned)c);
            last = (old + (unsigned)c == (unsigned)(npairs * rbs));
        }
        tile_cnt[t] = last;
    }
    __syncthreads();
    for (int t = 0; t < P.ntiles; ++t) {
        if (!tile_cnt[t]) continue;
        __threadfence();
        const int r0 = t * P.tile_rb * 32, r1 = min(P.Mpad, r0 + P.tile_rb * 32);
        for (int idx = tid; idx < (r1 - r0) * BT; idx += kThreads) {
            const int b = idx / (r1 - r0), r = r0 + idx % (r1 - r0);
            float *a = P.acc + (int64_t)b * P.Mpad + r;
            float v = __ldcg(a);
            __stcg(a, 0.f);
            if (r < P.M && b < P.nb) {
                if (P.y_fp32) ((float *)P.y)[(int64_t)b * P.ldy + r] = v;
                else ((__half *)P.y)[(int64_t)b * P.ldy + r] = __float2half_rn(v);
            }
        }
        if (tid == 0) P.tickets[t] = 0;
    }
}

// Test hook: build one table set exactly as the kernel does and write it out as [32][256] fp32.
__global__ void __launch_bounds__(kThreads, 1)
fluxbin_debug_tables_kernel(const uint8_t *pair_desc, const uint16_t *x, float *out)
{
    extern __shared__ __align__(16) uint8_t smem[];
    float *abuf = (float *)smem;
    const uint32_t base = (uint32_t)__cvta_generic_to_shared(smem);
    if (base + kSmallBytes > kTabBase) return;
    build_tables<1>(pair_desc, x, 0, 1, abuf);
    for (int i = threadIdx.x; i < 32 * 256; i += kThreads) {
        uint32_t sigma = i >> 8, p = i & 255;
        out[i] = *(const float *)(smem + ((TabCfg<1>::lane_const(sigma) | (p << 8)) - base));
    }
}

// Shared-window address at which dynamic shared memory starts for these kernels.
__global__ void fluxbin_smem_base_kernel(uint32_t *out)
{
    extern __shared__ __align__(16) uint8_t smem[];
    if (threadIdx.x == 0) *out = (uint32_t)__cvta_generic_to_shared(smem);
}

// dynamic shared memory to request: everything up to the end of the tables, as if the window began at 0
template <int BT> constexpr size_t smem_bytes() { return kTabBase + TabCfg<BT>::kTableBytes; }

} // namespace fbk
