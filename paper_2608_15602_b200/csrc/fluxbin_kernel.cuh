// FluxBin decode linear layer: the LUT GEMV kernel for sm_100a (no tensor cores: the path is a
// table-lookup GEMV bound by HBM and by the shared-memory lookup rate).
//
// One launch runs a list of layers ("entries": one for fluxbin_linear, many for a plan).  Persistent
// CTAs, several per SM.  The work of an entry is its list of items (pair, row block): a pair is one
// table set (32 tables = two units of 16 sub-vectors), a row block is 32 output rows.  The items
// of all entries, in order, are cut into equal contiguous shares (by cost), so a CTA builds the
// tables of one or two pairs (stage (i), Eq. 14, column scale fused per Eq. 11) and streams the
// weight bytes of a long run of rows through them (stage (ii), Eq. 15).  Row scales are applied
// per (row, segment) in registers and the per-row partial sums of this K slice are added to an
// fp32 accumulator in global memory (stage (iii)); the CTA that completes a tile of rows -- found
// with one arrival counter per tile, never by waiting -- converts the tile to the output type and
// re-zeroes the accumulator.  With many entries in one launch the start-up and reduction tails of
// one layer overlap the streaming of the next.
//
// Weight stream: every item is one contiguous block of memory.  A lane pulls its 32 weight bytes
// and its row scales straight into registers with 128-bit loads (staging them in shared memory
// would add traffic to the port the lookups saturate); L2 prefetches a trip or two ahead make
// those loads find their lines in L2.
//
// Shared-memory table layout: entry p of table slot sigma lives at  kTabBase + p*256 + sigma*E for
// entries of E = 4 or 8 bytes (the batch vectors of a launch side by side: 1 or 2 in fp32, 2 or 4 in
// fp16); 16-byte entries (4 vectors in fp32, 8 in fp16) put slots 16..31 into a second 64 KB half.
// A lane at step s reads slot lane ^ s, so the 32 lanes of a warp
// always hit 32 different slots: every lookup is bank-conflict free by construction, and the
// packer has stored each lane's weight bytes in exactly that order, so the byte of step s sits at
// a compile-time position.  In every mode the whole address is formed by ONE byte-permute (table
// index into byte 1, the lane's pre-packed slot offset into byte 0) and the table base rides in
// the load's immediate: 3 instructions per lookup and vector at batch 1 (PRMT, LDS, FADD).
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <type_traits>

#include "fluxbin_layout.h"

namespace fbk {

// The template parameter BT of everything below is a launch MODE: 1, 2 or 4 = that many batch vectors per
// launch with fp32 table entries (the precision the paper's shared-memory model states); 16 + n (n = 2, 4, 8)
// = n batch vectors with fp16 table entries, two vectors per 32-bit word -- half the shared-memory bytes per
// lookup, which is what bounds the batched path.  Sums still accumulate in fp32.  32 + n (n = 1, 2, 4) = n batch
// vectors with fp32 entries and sub-vectors of mu = 4 columns (the paper's sub-vector-size study): every byte of
// weight bits then indexes two 16-entry tables (its low and its high four columns) instead of one 256-entry table,
// so a table set (256 columns) shrinks from 32 KB to 4 KB per vector and the lookups double.  The packed layer is the same.
__host__ __device__ constexpr int nvec(int BT) { return BT & 15; }               // batch vectors per launch
__host__ __device__ constexpr bool half_tables(int BT) { return (BT & 16) != 0; }
__host__ __device__ constexpr bool mu4(int BT) { return (BT & 32) != 0; }
__host__ __device__ constexpr int geom(int BT) { return half_tables(BT) ? nvec(BT) / 2 : nvec(BT); }   // 32-bit words per table entry

// Threads per CTA: 8 warps with 4- or 8-byte entries (3 or 2 CTAs per SM); with 16-byte entries the
// tables fill 128 KB, one CTA owns the SM and runs 16 warps.
template <int BT> struct Cfg {
    static constexpr int kThreads = (geom(BT) == 4) ? 512 : 256;
    static constexpr int kWarps = kThreads / 32;
    static constexpr int kMinBlocks = (geom(BT) == 4) ? 1 : (geom(BT) == 2) ? 2 : 3;
};
constexpr int kMaxTiles = 1024;
constexpr int kDepth = 2;    // register sets (items in flight per warp) in the main loop
// The two-vector kernel runs 2 CTAs per SM (its tables are twice as large), so a thread may hold 128
// registers and fewer warps cover the load latency: it keeps more items in flight per warp
// (measured at batch 2 on a 16-layer stack: depth 2 3.49 TB/s, depth 3 3.56, depth 4 3.38).
constexpr int kDepth2 = 3;
constexpr int kDepth4 = 2;   // 16-byte entries: one CTA of 16 warps per SM
template <int BT> struct DepthFor { static constexpr int value = geom(BT) == 4 ? kDepth4 : geom(BT) == 2 ? kDepth2 : kDepth; };
// L2 prefetch distance in loop trips (one trip = kDepth items per warp).  Measured: 1 trip 5.40 TB/s,
// 2 trips 5.26, 3 trips 4.21, 8 trips 3.58 in a stripped copy of the loop -- far prefetches compete with
// the demand loads instead of helping them.
constexpr int kPrefetchTrips = 1;

// One layer of a launch.
struct LinearEntry {
    const uint8_t *packed;
    const uint16_t *x;       // [B][ldx] fp16
    void *y;                 // [B][ldy] fp16 or fp32
    float *acc;              // [BT][Mpad] split-K accumulators, zero on entry and on exit
    unsigned *tickets;       // [ntiles] arrival counters, zero on entry and on exit (shared by the two layers of a gated pair)
    long long ldx, ldy;
    float *acc2;             // gated pair: the partner layer's accumulators, else nullptr
    unsigned long long off_coldesc, off_items[2];
    int M, N, Kb, nrb;       // rows are padded to Mpad = nrb * 32
    int npairs[2];
    int arrivals;            // (pair, row block) items that complete one row block: npairs[0] + npairs[1], plus the partner's in a gated pair
    int tile_rb, ntiles;
    int flags;               // bits 0..7: table slots of the last salient pair (32; 16 or 8: stored narrow); bits 8..9: role in a
                             // gated pair (0 none, 1 gate: y = silu(this) * partner, 2 up: y = silu(partner) * this)
    __host__ __device__ int mpad() const { return nrb * 32; }
    __host__ __device__ int sal_last_w() const { return flags & 0xff; }
    __host__ __device__ int role() const { return (flags >> 8) & 3; }
};

// Where a share of a launch begins: layer `entry`, work item `item` of it (a work item is one row block of one
// work pair -- NP pairs of the global region walked together, or one salient pair -- numbered pair-major:
// global region first).  The host cuts the cost line of the launch once and hands every share its bounds.
struct ShareCut {
    int entry, item;
};

constexpr int kMaxSingleShares = 512;      // shares (= CTAs) of a launch whose cuts travel in the parameters

struct LaunchParams {
    const LinearEntry *table;   // device table of n entries; nullptr: the single entry below
    const ShareCut *cuts;       // device [nshares + 1] with a table; nullptr: single_cut below
    LinearEntry single;
    int n;
    int nb;                     // live batch rows (<= BT)
    int y_fp32;
    int nshares;                // grid size + number of small shares drawn dynamically after it
    unsigned *counters;         // [2] share counter and exit counter, zero on entry and on exit
#ifdef FB_TRACE
    int trace_slot;             // instrumented build: which of the eight trace buffers this launch writes
#endif
    int single_cut[kMaxSingleShares + 1];    // first work item of share s of the single entry; [nshares] = all items
};

// The tables start at this shared-window address.  It is a compile-time constant so that it can
// ride in the immediate field of every table load; dynamic shared memory starts below it (1 KB is
// reserved by the system at the bottom of the window; the host probes the actual start once).
constexpr uint32_t kTabBase = 0x800u;

template <int BT> struct TabCfg {
    static constexpr int kTableBytes = (geom(BT) == 4) ? 131072 : 65536;
    // scale-fusion scratch (for two table sets when two fit side by side: 4-byte entries), tile counters
    // (+ count of completed tiles), work range, copy of the current entry
    static constexpr int kScratchFloats = 256 * nvec(BT) * (geom(BT) == 1 ? 2 : 1);
    static constexpr int kSmallBytes = kScratchFloats * 4 + (kMaxTiles + 4) * 4 + 32 + 128;
    // offset of slot sigma from the table base at step 0; entry p adds p << 8.
    // lane_const(lane ^ s) == lane_const(lane) ^ lane_const(s)
    __host__ __device__ static constexpr uint32_t lane_const(uint32_t sigma)
    {
        return geom(BT) == 1 ? sigma * 4u : geom(BT) == 2 ? sigma * 8u : ((sigma & 15u) * 16u) | ((sigma >> 4) << 16);
    }
};

// W = steps (table slots) per item: 32, or 16 / 8 for the narrow last pair of a salient region
template <int SPS, int W = 32> struct ItemBytes { static constexpr int value = 32 * W + 64 * (W / SPS); };
static_assert(ItemBytes<16>::value == FB_ITEM_BITS_BYTES + 64 * 2, "full items: 1024 bytes of weight bits");

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

template <int BT> struct Vec { float v[nvec(BT)]; };

// HALF selects the table set inside the 256-byte p-rows: slots 0..31 or (4-byte entries only) slots 32..63.
// HI (mu = 4 only) selects the tables of a byte's high four columns: p-rows 16..31 instead of 0..15.
template <int BT, int HALF, int HI = 0> __device__ __forceinline__ Vec<BT> lds_entry(uint32_t addr)
{
    Vec<BT> r;
    // addr is an offset from the table base; base, half and row offset ride in the immediate
    constexpr uint32_t kBase = kTabBase + HI * (16u << 8);
    if constexpr (geom(BT) == 1) asm volatile("ld.shared.f32 %0, [%1+%2];" : "=f"(r.v[0]) : "r"(addr), "n"(kBase + HALF * 128));
    else if constexpr (geom(BT) == 2) asm volatile("ld.shared.v2.f32 {%0,%1}, [%2+%3];" : "=f"(r.v[0]), "=f"(r.v[1]) : "r"(addr), "n"(kBase));
    else asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4+%5];" : "=f"(r.v[0]), "=f"(r.v[1]), "=f"(r.v[2]), "=f"(r.v[3]) : "r"(addr), "n"(kBase));
    return r;
}

// fp16 tables: the geom(BT) words of one entry, two batch vectors per word (vector 2i in the low half of word i)
template <int BT, int HALF> __device__ __forceinline__ void lds_entry_h(uint32_t addr, uint32_t (&w)[geom(BT)])
{
    if constexpr (geom(BT) == 1) asm volatile("ld.shared.b32 %0, [%1+%2];" : "=r"(w[0]) : "r"(addr), "n"(kTabBase + HALF * 128));
    else if constexpr (geom(BT) == 2) asm volatile("ld.shared.v2.b32 {%0,%1}, [%2+%3];" : "=r"(w[0]), "=r"(w[1]) : "r"(addr), "n"(kTabBase));
    else asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4+%5];" : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "r"(addr), "n"(kTabBase));
}

// lo += low half of h2, hi += high half of h2: fp16 addends, fp32 sums (one instruction each on sm_100)
__device__ __forceinline__ void add_h2(float &lo, float &hi, uint32_t h2)
{
    asm("{\n\t.reg .b16 l, h;\n\tmov.b32 {l, h}, %2;\n\tadd.rn.f32.f16 %0, l, %0;\n\tadd.rn.f32.f16 %1, h, %1;\n\t}"
        : "+f"(lo), "+f"(hi) : "r"(h2));
}

// NV fp32 values rounded to fp16 (to nearest even) and stored as NV/2 words at byte `off` of the entry at addr
template <int NV> __device__ __forceinline__ void sts_entry_h(uint32_t addr, const float *v)
{
    uint32_t w[NV / 2];
#pragma unroll
    for (int i = 0; i < NV / 2; ++i) asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(w[i]) : "f"(v[2 * i + 1]), "f"(v[2 * i]));
    if constexpr (NV == 2) asm volatile("st.shared.b32 [%0+%2], %1;" ::"r"(addr), "r"(w[0]), "n"(kTabBase) : "memory");
    else asm volatile("st.shared.v2.b32 [%0+%3], {%1,%2};" ::"r"(addr), "r"(w[0]), "r"(w[1]), "n"(kTabBase) : "memory");
}

// the NV batch vectors of one entry at table offset addr
template <int NV> __device__ __forceinline__ void sts_entry(uint32_t addr, const float *v)
{
    if constexpr (NV == 1) asm volatile("st.shared.f32 [%0+%2], %1;" ::"r"(addr), "f"(v[0]), "n"(kTabBase) : "memory");
    else if constexpr (NV == 2) asm volatile("st.shared.v2.f32 [%0+%3], {%1,%2};" ::"r"(addr), "f"(v[0]), "f"(v[1]), "n"(kTabBase) : "memory");
    else asm volatile("st.shared.v4.f32 [%0+%5], {%1,%2,%3,%4};" ::"r"(addr), "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "n"(kTabBase) : "memory");
}

// PRMT with the full selector: bit 3 of a nibble replicates the sign bit of the selected byte
// (the __byte_perm intrinsic masks that bit away, so the instruction is spelled out).
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel)
{
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

// One 128-byte line into L2, under a predicate (no branch, no reconvergence point in the caller's loop).
__device__ __forceinline__ void prefetch_line_if(const void *p, bool pred)
{
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.b32 q, %1, 0;\n\t@q prefetch.global.L2 [%0];\n\t}" ::"l"(p), "r"((uint32_t)pred) : "memory");
}

// fp32 add into the split-K accumulator (global memory by contract).  Spelled out as a reduction on the
// global window: through a generic pointer the compiler emits an address-space check with a divergence
// barrier, a vote and a branch around every atomic.
__device__ __forceinline__ void red_add_f32(float *p, float v)
{
    asm volatile("red.global.add.f32 [%0], %1;" ::"l"(__cvta_generic_to_global(p)), "f"(v) : "memory");
}

// One bulk request that pulls `bytes` (a multiple of 16) starting at p into L2.
__device__ __forceinline__ void prefetch_l2(const void *p, uint32_t bytes)
{
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p), "r"(bytes) : "memory");
}


// ---------------------------------------------------------------------------------------------
// Stage (i): LUT building with scale fusion (Eq. 14 with a_n = x[col_n] * alpha_c[col_n], Eq. 11;
// for salient tables col_n = sal_idx[v] and alpha = gathered scale, Eq. 13).
// abuf: shared scratch of 32*8*BT floats.  build_tables ends with the tables visible to the whole CTA.
// col0_a / col0_b: first column of the pair's two units for a global pair, -1 for a salient pair.
// ---------------------------------------------------------------------------------------------
// The two values a thread contributes to a table set: x of its column (per batch vector) and the
// fused column scale.
template <int BT> struct BuildInput {
    float xv[nvec(BT)];
    uint32_t e;        // {u16 column, fp16 alpha}
};

// The static half of a table set's inputs: {u16 column, fp16 alpha} of (slot tid/8, n tid%8) from the pair's
// column table.  It belongs to the packed layer, so it may be requested before the launch's predecessor is done.
template <int BT>
__device__ __forceinline__ void fetch_build_desc(BuildInput<BT> &in, const uint8_t *pair_desc)
{
    const int tid = threadIdx.x;
    if (Cfg<BT>::kThreads > 256 && tid >= 256) return;      // one thread per table column
    in.e = __ldg((const uint32_t *)pair_desc + tid);
}

// The activations of the thread's column.  For a global pair the column is known from the pair's position, so
// this load does not wait for the column table; for a salient pair it is the column the table names.
template <int BT>
__device__ __forceinline__ void fetch_build_x(BuildInput<BT> &in, const uint16_t *x, int64_t ldx, int nb, int col0_a, int col0_b,
                                              int ncols)
{
    const int tid = threadIdx.x;
    if (Cfg<BT>::kThreads > 256 && tid >= 256) return;
    if (col0_a >= 0) {       // first unit of the pair: slots 0..15, second unit: slots 16..31
        const uint32_t col = (uint32_t)(tid < 128 ? col0_a : col0_b) + (uint32_t)(tid & 127);
        const bool live = col < (uint32_t)ncols;          // padded columns carry alpha = 0
#pragma unroll
        for (int b = 0; b < nvec(BT); ++b) in.xv[b] = (b < nb && live) ? h2f(__ldg(x + (int64_t)b * ldx + col)) : 0.f;
    } else {
        const uint32_t col = in.e & 0xffffu;
#pragma unroll
        for (int b = 0; b < nvec(BT); ++b) in.xv[b] = (b < nb) ? h2f(__ldg(x + (int64_t)b * ldx + col)) : 0.f;
    }
}

template <int BT>
__device__ __forceinline__ void fetch_build_input(BuildInput<BT> &in, const uint8_t *pair_desc, const uint16_t *x,
                                                  int64_t ldx, int nb, int col0_a, int col0_b, int ncols)
{
    fetch_build_desc<BT>(in, pair_desc);
    fetch_build_x<BT>(in, x, ldx, nb, col0_a, col0_b, ncols);
}

// Scratch index of a_n of table slot `slot`, batch vector b: rows of 32 slots, rotated by 4n so that both
// the writers (8 n x 4 slots per warp) and the readers (32 slots per warp, one n) touch 32 different banks.
template <int BT> __device__ __forceinline__ int abuf_index(int slot, int n, int b)
{
    return (n * nvec(BT) + b) * 32 + ((slot + 4 * n) & 31);
}

// Scale fusion (Eq. 11): a_n = x * alpha of the thread's table column into the scratch.
template <int BT>
__device__ __forceinline__ void stage_build_input(const BuildInput<BT> &in, float *abuf)
{
    const int tid = threadIdx.x;
    constexpr int NV = nvec(BT);
    if (Cfg<BT>::kThreads == 256 || tid < 256) {
        const float al = h2f(in.e >> 16);
#pragma unroll
        for (int b = 0; b < NV; ++b) abuf[abuf_index<BT>(tid >> 3, tid & 7, b)] = in.xv[b] * al;   // exact in fp32: two 11-bit significands
    }
}

// All 256 entries of the 32 tables of one table set from the staged a_n (Eq. 14); the caller puts a barrier
// between staging and this, and one after it.
template <int BT>
__device__ __forceinline__ void enumerate_tables(const float *abuf, uint32_t half_off)
{
    const int tid = threadIdx.x;
    constexpr int NV = nvec(BT);
    const int lane = tid & 31, warp = tid >> 5;
    if constexpr (mu4(BT)) {
        // mu = 4: two 16-entry tables per slot -- p-rows 0..15 index columns 0..3 of the slot's eight, p-rows 16..31
        // columns 4..7 (Eq. 14 with mu = 4); a warp fills whole p-rows, one entry (all vectors) per lane and row.
        static_assert(!half_tables(BT) && NV <= 4, "mu = 4 runs with fp32 entries");
        float a[8][NV];
#pragma unroll
        for (int n = 0; n < 8; ++n)
#pragma unroll
            for (int b = 0; b < NV; ++b) a[n][b] = abuf[abuf_index<BT>(lane, n, b)];
#pragma unroll 1
        for (int p = warp; p < 32; p += Cfg<BT>::kWarps) {
            float v[NV];
#pragma unroll
            for (int b = 0; b < NV; ++b) {
                float sum = 0.f;
#pragma unroll
                for (int n = 3; n >= 0; --n) {
                    const float an = (p & 16) ? a[4 + n][b] : a[n][b];
                    sum += ((p >> n) & 1) ? an : -an;
                }
                v[b] = sum;
            }
            sts_entry<NV>(half_off | TabCfg<BT>::lane_const((uint32_t)lane) | ((uint32_t)p << 8), v);
        }
        return;
    }
    // EB entries at a time: the high index bits fix a base value, the low LB bits are enumerated by
    // doubling (entry p | 2^n = entry p + 2 a_n), one add per entry.  Up to four batch vectors of an entry are
    // stored with one instruction (with four, blocks of 8 entries keep the registers in bounds).  With eight
    // vectors (fp16 entries) half of the warps fill vectors 0..3 and half vectors 4..7 of all entries -- and
    // within a warp lanes 8..15 and 24..31 take the other group than lanes 0..7 and 16..23, so that the 8-byte
    // stores of a warp, 16 bytes apart, cover all 32 banks (two wavefronts per 256 bytes instead of four).
    constexpr int PV = NV < 4 ? NV : 4;                // vectors per thread
    constexpr int NG = NV / PV;                        // groups of vectors (1 or 2)
    constexpr int PW = 256 / (Cfg<BT>::kWarps / NG);   // table entries per warp: p = (warp % (kWarps/NG))*PW + ...
    constexpr int LB = (PV == 4) ? 3 : 4, EB = 1 << LB;
    static_assert(PW % EB == 0, "a warp enumerates whole blocks of entries");
    const int wl = NG == 1 ? warp : warp % (Cfg<BT>::kWarps / NG);
    const int b0 = NG == 1 ? 0 : PV * ((warp / (Cfg<BT>::kWarps / NG)) ^ ((lane >> 3) & 1));
    float a[8][PV];
#pragma unroll
    for (int n = 0; n < 8; ++n)
#pragma unroll
        for (int b = 0; b < PV; ++b) a[n][b] = abuf[abuf_index<BT>(lane, n, b0 + b)];
#pragma unroll 1
    for (int p0 = wl * PW; p0 < (wl + 1) * PW; p0 += EB) {
        float v[EB][PV];
#pragma unroll
        for (int b = 0; b < PV; ++b) {
            float base = 0.f;
#pragma unroll
            for (int n = 7; n >= LB; --n) base += ((p0 >> n) & 1) ? a[n][b] : -a[n][b];
#pragma unroll
            for (int n = LB - 1; n >= 0; --n) base -= a[n][b];
            v[0][b] = base;
#pragma unroll
            for (int n = 0; n < LB; ++n)
#pragma unroll
                for (int q = 0; q < (1 << n); ++q) v[q | (1 << n)][b] = v[q][b] + 2.f * a[n][b];
        }
#pragma unroll
        for (int q = 0; q < EB; ++q) {
            const uint32_t addr = half_off | TabCfg<BT>::lane_const((uint32_t)lane) | ((uint32_t)(p0 + q) << 8);
            if constexpr (half_tables(BT)) sts_entry_h<PV>(addr + 2u * (uint32_t)b0, v[q]);    // rounded once, from the fp32 sum
            else sts_entry<PV>(addr, v[q]);
        }
    }
}

// One table set; ends with the tables visible to the whole CTA.
template <int BT>
__device__ __forceinline__ void build_tables(const BuildInput<BT> &in, float *abuf, uint32_t half_off = 0)
{
    stage_build_input<BT>(in, abuf);
    __syncthreads();
    enumerate_tables<BT>(abuf, half_off);
    __syncthreads();
}

// Two table sets side by side (4-byte entries: slots 0..31 and 32..63 of the 256-byte rows) behind one pair of barriers.
template <int BT>
__device__ __forceinline__ void build_tables2(const BuildInput<BT> &in_a, const BuildInput<BT> &in_b, float *abuf)
{
    static_assert(geom(BT) == 1, "two table sets side by side need 4-byte entries");
    stage_build_input<BT>(in_a, abuf);
    stage_build_input<BT>(in_b, abuf + 256 * nvec(BT));
    __syncthreads();
    enumerate_tables<BT>(abuf, 0u);
    enumerate_tables<BT>(abuf + 256 * nvec(BT), 128u);
    __syncthreads();
}

// ---------------------------------------------------------------------------------------------
// Stage (ii)+(iii) for one run of row blocks of one pair.
// SPS = sub-vectors per row-scale segment (16: one scale per unit and row; 1: one per sub-vector).
// ---------------------------------------------------------------------------------------------
template <int SPS, int W = 32> struct ItemRegs {
    static constexpr int kSc = (W / SPS + 1) / 2;     // 32-bit words of row scales per lane
    uint4 b0, b1;                         // weight bytes of steps 0..15 / 16..31
    uint32_t sc[kSc];
};

// pl = item + lane * min(W, 16) (weight bytes), ps = item + 32 * W + lane * (scale bytes per lane and plane, at
// most 16); `off` is a compile-time byte offset added to both (the stride to a later item).
template <int SPS, int W = 32> __device__ __forceinline__ void load_item(ItemRegs<SPS, W> &r, const uint8_t *pl, const uint8_t *ps, int off)
{
    constexpr int kSc = ItemRegs<SPS, W>::kSc;
    if constexpr (W == 8) { const uint2 t = ldg_stream_v2(pl + off); r.b0.x = t.x; r.b0.y = t.y; }
    else r.b0 = ldg_stream_v4(pl + off);
    if constexpr (W == 32) r.b1 = ldg_stream_v4(pl + off + 512);
    if constexpr (kSc == 1) r.sc[0] = ldg_stream_u32(ps + off);
    else if constexpr (kSc == 2) { uint2 t = ldg_stream_v2(ps + off); r.sc[0] = t.x; r.sc[1] = t.y; }
    else {
#pragma unroll
        for (int q = 0; q < kSc / 4; ++q) {               // planes of 8 halves per lane
            uint4 t = ldg_stream_v4(ps + off + q * 512);
            r.sc[4 * q] = t.x; r.sc[4 * q + 1] = t.y; r.sc[4 * q + 2] = t.z; r.sc[4 * q + 3] = t.w;
        }
    }
}

// The three parts of an item separately (SPS >= 2), each into the registers its predecessor's lookups have freed.
template <int SPS> __device__ __forceinline__ void load_scales(ItemRegs<SPS> &r, const uint8_t *ps, int off)
{
    if constexpr (SPS == 16) r.sc[0] = ldg_stream_u32(ps + off);
    else if constexpr (SPS == 8) { uint2 t = ldg_stream_v2(ps + off); r.sc[0] = t.x; r.sc[1] = t.y; }
    else { uint4 t = ldg_stream_v4(ps + off); r.sc[0] = t.x; r.sc[1] = t.y; r.sc[2] = t.z; r.sc[3] = t.w; }
}

// Lane constant of the lookup address.  BT == 1: one register holding, byte by byte, the slot offsets
// (lane ^ k) * 4 of steps k = 0..3, so that PRMT can drop one into byte 0 of the address; the offsets
// of steps 4q + k differ from these by an XOR with 16q in every byte ((lane ^ (4q + k)) * 4 ==
// ((lane ^ k) * 4) ^ 16q), one LOP per group of four lookups instead of eight live registers.
// BT == 2: the slot offsets (lane ^ s) * 8 reach 248, so a byte of them cannot double as the zero
// fill of the upper address bytes; each register holds the offsets of two steps and two zero bytes,
// and with 128 registers per thread all sixteen stay resident (no LOP at all).
template <int BT> struct LaneAddr;
template <> struct LaneAddr<1> {
    uint32_t c0;
    __device__ __forceinline__ void init(int lane)
    {
        uint32_t v = 0;
#pragma unroll
        for (int k = 0; k < 4; ++k) v |= (uint32_t)(((lane ^ k) * 4) & 0xff) << (8 * k);
        c0 = v;
        asm volatile("" : "+r"(c0));      // keep it in its register: recomputing it per item costs more
    }
    // address of the lookup of step s: byte 1 = table index (byte s%4 of w), byte 0 = slot offset
    __device__ __forceinline__ uint32_t addr(int s, uint32_t w) const     // s: compile-time after unrolling
    {
        const uint32_t k = (uint32_t)s & 3u;
        return prmt(w, c0 ^ (0x10101010u * (uint32_t)(s >> 2)), ((0xCu | k) << 12) | ((0xCu | k) << 8) | (k << 4) | (4u | k));
    }
};
template <> struct LaneAddr<2> {
    uint32_t c[16];
    __device__ __forceinline__ void init(int lane)
    {
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            c[i] = (uint32_t)((lane ^ (2 * i)) * 8) | ((uint32_t)((lane ^ (2 * i + 1)) * 8) << 8);
            asm volatile("" : "+r"(c[i]));
        }
    }
    __device__ __forceinline__ uint32_t addr(int s, uint32_t w) const
    {
        const uint32_t k = (uint32_t)s & 3u, j = (uint32_t)s & 1u;
        return prmt(w, c[s >> 1], (6u << 12) | (6u << 8) | (k << 4) | (4u | j));
    }
};

// BT == 4: 16-byte entries; slots 0..15 and 16..31 live in two 64 KB halves, so byte 2 of the address
// carries the half ((lane ^ s) >> 4, the same for steps 2i and 2i + 1) and byte 3 is zero.
template <> struct LaneAddr<4> {
    uint32_t c[16];
    __device__ __forceinline__ void init(int lane)
    {
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const uint32_t s0 = (uint32_t)(lane ^ (2 * i)), s1 = (uint32_t)(lane ^ (2 * i + 1));
            c[i] = ((s0 & 15u) * 16u) | (((s1 & 15u) * 16u) << 8) | ((s0 >> 4) << 16);
            asm volatile("" : "+r"(c[i]));
        }
    }
    __device__ __forceinline__ uint32_t addr(int s, uint32_t w) const
    {
        const uint32_t k = (uint32_t)s & 3u, j = (uint32_t)s & 1u;
        return prmt(w, c[s >> 1], (7u << 12) | (6u << 8) | (k << 4) | (4u | j));
    }
};

// the table geometry of the fp16 modes is that of the fp32 mode with the same entry size
template <> struct LaneAddr<16 + 2> : LaneAddr<1> {};
template <> struct LaneAddr<16 + 4> : LaneAddr<2> {};
template <> struct LaneAddr<16 + 8> : LaneAddr<4> {};
// mu = 4: the same slots, the table index is a nibble of the weight byte (masked out before the PRMT)
template <> struct LaneAddr<32 + 1> : LaneAddr<1> {};
template <> struct LaneAddr<32 + 2> : LaneAddr<2> {};
template <> struct LaneAddr<32 + 4> : LaneAddr<4> {};

// Two alternating partial sums per vector shorten the dependency chain of a segment's adds; with four or more
// vectors the adds of one lookup already space out each vector's chain (+1-5 % without the split there).
constexpr int kSplitBelowVectors = 4;
template <int SPS, int BT, int HALF = 0, int W = 32>
__device__ __forceinline__ void compute_item(const ItemRegs<SPS, W> &r, const LaneAddr<BT> &la, float (&out)[nvec(BT)])
{
    constexpr int NSEG = W / SPS;
    constexpr int NV = nvec(BT);
    const uint32_t w[8] = {r.b0.x, r.b0.y, r.b0.z, r.b0.w, r.b1.x, r.b1.y, r.b1.z, r.b1.w};
#pragma unroll
    for (int b = 0; b < NV; ++b) out[b] = 0.f;
#pragma unroll
    for (int j = 0; j < NSEG; ++j) {
        float seg[NV];
        {
            // (a packed add.f32x2 for two lookups was measured 2 % slower: the pairing costs a MOV per lookup)
            float s0[NV], s1[NV];
#pragma unroll
            for (int b = 0; b < NV; ++b) { s0[b] = 0.f; s1[b] = 0.f; }
#pragma unroll
            for (int q = 0; q < SPS; ++q) {
                const int s = j * SPS + q;
                if constexpr (mu4(BT)) {
                    // the byte's low and high four columns: two lookups (the masks are shared by the four steps of a word)
                    const uint32_t lo = w[s >> 2] & 0x0f0f0f0fu, hi = (w[s >> 2] >> 4) & 0x0f0f0f0fu;
                    const Vec<BT> e0 = lds_entry<BT, HALF, 0>(la.addr(s, lo));
                    const Vec<BT> e1 = lds_entry<BT, HALF, 1>(la.addr(s, hi));
#pragma unroll
                    for (int b = 0; b < NV; ++b) {
                        s0[b] += e0.v[b];
                        if (NV < kSplitBelowVectors) s1[b] += e1.v[b]; else s0[b] += e1.v[b];
                    }
                    continue;
                }
                const uint32_t addr = la.addr(s, w[s >> 2]);
                if constexpr (half_tables(BT)) {
                    uint32_t e[geom(BT)];
                    lds_entry_h<BT, HALF>(addr, e);
#pragma unroll
                    for (int i = 0; i < geom(BT); ++i) {
                        if ((q & 1) && NV < kSplitBelowVectors) add_h2(s1[2 * i], s1[2 * i + 1], e[i]); else add_h2(s0[2 * i], s0[2 * i + 1], e[i]);
                    }
                } else {
                    Vec<BT> e = lds_entry<BT, HALF>(addr);
#pragma unroll
                    for (int b = 0; b < NV; ++b) {
                        if ((q & 1) && NV < kSplitBelowVectors) s1[b] += e.v[b]; else s0[b] += e.v[b];
                    }
                }
            }
#pragma unroll
            for (int b = 0; b < NV; ++b) seg[b] = (NV >= kSplitBelowVectors) ? s0[b] : s0[b] + s1[b];
        }
        float scale = h2f((r.sc[j >> 1] >> ((j & 1) * 16)) & 0xffffu);
#pragma unroll
        for (int b = 0; b < NV; ++b) out[b] = fmaf(scale, seg[b], out[b]);
    }
}

// Half an item (steps 16H .. 16H+15, the weight bytes of one 128-bit load) for one batch vector: adds the
// scaled segment sums of that half to out.  SPS >= 2.
template <int SPS, int HALF, int H>
__device__ __forceinline__ void compute_half(const uint4 &b, const uint32_t *sc, const LaneAddr<1> &la, float &out)
{
    static_assert(SPS >= 2 && SPS <= 16, "segments do not straddle the two halves");
    constexpr int NSEG_H = 16 / SPS;
    const uint32_t w[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
    for (int jj = 0; jj < NSEG_H; ++jj) {
        const int j = H * NSEG_H + jj;
        float s0 = 0.f, s1 = 0.f;
#pragma unroll
        for (int q = 0; q < SPS; ++q) {
            const int s = j * SPS + q;
            const float e = lds_entry<1, HALF>(la.addr(s, w[(s >> 2) & 3])).v[0];
            if (q & 1) s1 += e; else s0 += e;
        }
        const float scale = h2f((sc[j >> 1] >> ((j & 1) * 16)) & 0xffffu);
        out = fmaf(scale, s0 + s1, out);
    }
}

// The same for two batch vectors with fp16 table entries (one 32-bit word per lookup holds both).
template <int SPS, int HALF, int H>
__device__ __forceinline__ void compute_half_h2(const uint4 &b, const uint32_t *sc, const LaneAddr<1> &la, float &out0, float &out1)
{
    static_assert(SPS >= 2 && SPS <= 16, "segments do not straddle the two halves");
    constexpr int NSEG_H = 16 / SPS;
    const uint32_t w[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
    for (int jj = 0; jj < NSEG_H; ++jj) {
        const int j = H * NSEG_H + jj;
        float s0 = 0.f, s1 = 0.f, t0 = 0.f, t1 = 0.f;
#pragma unroll
        for (int q = 0; q < SPS; ++q) {
            const int s = j * SPS + q;
            uint32_t e[1];
            lds_entry_h<16 + 2, HALF>(la.addr(s, w[(s >> 2) & 3]), e);
            if (q & 1) add_h2(s1, t1, e[0]); else add_h2(s0, t0, e[0]);
        }
        const float scale = h2f((sc[j >> 1] >> ((j & 1) * 16)) & 0xffffu);
        out0 = fmaf(scale, s0 + s1, out0);
        out1 = fmaf(scale, t0 + t1, out1);
    }
}

template <int SPS, int BT, int W = 32>
__device__ __forceinline__ void finish_item(const ItemRegs<SPS, W> &r, const LaneAddr<BT> &la, float *accp, int Mpad)
{
    float out[nvec(BT)];
    compute_item<SPS, BT, 0, W>(r, la, out);
#pragma unroll
    for (int b = 0; b < nvec(BT); ++b) red_add_f32(accp + (int64_t)b * Mpad, out[b]);
}

// The first item of this warp's run, loaded ahead of the table build so that its latency hides
// behind the build (the weights do not depend on the activations).
template <int SPS, int BT>
__device__ __forceinline__ void preload_first(ItemRegs<SPS> &r, const uint8_t *pair_items, int rb_lo, int rb_hi)
{
    constexpr int IB = ItemBytes<SPS>::value;
    constexpr int SB = (SPS == 16) ? 4 : (SPS == 8) ? 8 : 16;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int first = rb_lo + warp;
    if (first >= rb_hi) return;
    const uint8_t *item = pair_items + (int64_t)first * IB;
    load_item<SPS>(r, item + lane * 16, item + FB_ITEM_BITS_BYTES + lane * SB, 0);
}

// Row blocks rb_lo + warp, + kWarps, ... of one pair.  kDepth register sets rotate so that the
// loads of the next kDepth-1 items are in flight while the current one is looked up (enough bytes
// in flight per SM to cover the L2 latency at full HBM rate).  A trip of the steady loop handles
// kDepth items with every address a pointer plus an immediate; each warp also bulk-prefetches,
// kPrefetchTrips trips ahead, its share of the kDepth*kWarps items the CTA reads per trip.
template <int SPS, int BT, int W = 32>
__device__ __forceinline__ void process_rows(const uint8_t *pair_items, int rb_lo, int rb_hi,
                                             const LaneAddr<BT> &la, float *acc, int Mpad,
                                             const ItemRegs<SPS, W> *pre = nullptr)   // pre: preload_first's result
{
    constexpr int IB = ItemBytes<SPS, W>::value;
    constexpr int kWarps = Cfg<BT>::kWarps;
    constexpr int STRIDE = kWarps * IB;                   // bytes between a warp's consecutive items
    constexpr int kSc = ItemRegs<SPS, W>::kSc;
    constexpr int SB = kSc == 1 ? 4 : kSc == 2 ? 8 : 16;  // scale bytes per lane (per plane)
    constexpr int D = (SPS == 1) ? 1 : DepthFor<BT>::value;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int first = rb_lo + warp;
    if (first >= rb_hi) return;
    const int n = (rb_hi - first + kWarps - 1) / kWarps;  // items of this warp
    const uint8_t *pl = pair_items + (int64_t)first * IB + lane * (W < 16 ? W : 16);
    const uint8_t *ps = pair_items + (int64_t)first * IB + 32 * W + lane * SB;
    // this warp's prefetch window inside the block of D*kWarps items the CTA consumes per trip
    const uint8_t *pp = pair_items + (int64_t)(rb_lo + D * warp) * IB + (int64_t)kPrefetchTrips * D * STRIDE;
    const uint8_t *pend = pair_items + (int64_t)rb_hi * IB;
    float *accp = acc + first * 32 + lane;

    ItemRegs<SPS, W> r[D];
#pragma unroll
    for (int d = 0; d < D - 1; ++d) {
        if (d == 0 && pre) r[0] = *pre;
        else if (d < n) load_item<SPS, W>(r[d], pl, ps, d * STRIDE);
    }
    // items t .. t+D-1 are looked up while items t+D-1 .. t+2D-2 are loaded (warp-uniform guards)
    for (int t = 0; t < n; t += D) {
        if (lane == 0 && pp + D * IB <= pend) prefetch_l2(pp, D * IB);
#pragma unroll
        for (int d = 0; d < D; ++d) {
            if (t + d + D - 1 < n) load_item<SPS, W>(r[(d + D - 1) % D], pl, ps, (d + D - 1) * STRIDE);
            if (t + d < n) finish_item<SPS, BT, W>(r[d], la, accp + d * (kWarps * 32), Mpad);
        }
        pl += D * STRIDE;
        ps += D * STRIDE;
        pp += D * STRIDE;
        accp += D * kWarps * 32;
    }
}

// The same for TWO pairs whose table sets are resident together (slots 0..31 and 32..63, 4-byte entries):
// for every row block the lane looks up the item of the first pair, then the item of the second
// (items_b = the second pair's items), adds the two row sums and issues ONE reduction -- half the
// atomic traffic and half the per-item bookkeeping.  One item is always in flight ahead.
// BT: 1 (one vector, fp32 entries) or 16 + 2 (two vectors, fp16 entries: the same 4-byte slots).
template <int SPS, int BT>
__device__ __forceinline__ void process_rows2(const uint8_t *items_a, const uint8_t *items_b, int rb_lo, int rb_hi,
                                              const LaneAddr<1> &la, float *acc, int Mpad)
{
    static_assert(geom(BT) == 1, "two table sets side by side need 4-byte entries");
    // lookups of one 128-bit half of an item, added to the row sums of the batch vectors
    auto half = [&](auto set, auto h, const uint4 &b, const uint32_t *sc, float &o0, float &o1) {
        if constexpr (BT == 1) compute_half<SPS, decltype(set)::value, decltype(h)::value>(b, sc, la, o0);
        else compute_half_h2<SPS, decltype(set)::value, decltype(h)::value>(b, sc, la, o0, o1);
    };
    using I0 = std::integral_constant<int, 0>;
    using I1 = std::integral_constant<int, 1>;
    constexpr int IB = ItemBytes<SPS>::value;
    constexpr int kWarps = Cfg<1>::kWarps;
    constexpr int STRIDE = kWarps * IB;
    constexpr int SB = (SPS == 16) ? 4 : (SPS == 8) ? 8 : 16;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int first = rb_lo + warp;
    if (first >= rb_hi) return;
    const int n = (rb_hi - first + kWarps - 1) / kWarps;
    const int64_t o_l = (int64_t)first * IB + lane * 16, o_s = (int64_t)first * IB + FB_ITEM_BITS_BYTES + lane * SB;
    const uint8_t *pla = items_a + o_l, *psa = items_a + o_s;
    const uint8_t *plb = items_b + o_l, *psb = items_b + o_s;
    // lanes 0..8 and 9..17 of every warp prefetch, line by line, the warp's own item of the trip
    // kPrefetchTrips + 1 ahead in the first and the second pair (one ordinary instruction per trip: the bulk
    // prefetch is a uniform-datapath instruction and costs a lane-by-lane loop when its address is per lane)
    static_assert(IB % 128 == 0 && IB / 128 <= 16, "an item is at most 16 lines");
    constexpr int LPI = IB / 128;
    const uint8_t *pp = (lane < LPI ? items_a : items_b) + (int64_t)first * IB + (int64_t)(kPrefetchTrips + 1) * STRIDE +
                        (lane < LPI ? lane : lane - LPI) * 128;
    float *accp = acc + first * 32 + lane;

    // Both items of the current row block are in registers (or on their way) at the top of a trip; each
    // 128-bit half of the next row block's items is requested as soon as the lookups of the half it
    // replaces are done, so a load has 1.5 item times to arrive instead of one, with no extra registers.
    // The last row block is peeled off: the steady state has no guards in it, and the prefetch is one
    // predicated instruction (guards cost about 20 instructions per item in moves, predicates and branches).
    ItemRegs<SPS> ra, rb;
    load_item<SPS>(ra, pla, psa, 0);
    load_item<SPS>(rb, plb, psb, 0);
    const int n_pf = lane < 2 * LPI ? n - (kPrefetchTrips + 1) : 0;      // trips in which this lane prefetches
    for (int t = 0; t < n - 1; ++t) {
        prefetch_line_if(pp, t < n_pf);
        float o = 0.f, o1 = 0.f;
        half(I0{}, I0{}, ra.b0, ra.sc, o, o1);
        ra.b0 = ldg_stream_v4(pla + STRIDE);
        half(I0{}, I1{}, ra.b1, ra.sc, o, o1);
        ra.b1 = ldg_stream_v4(pla + STRIDE + 512);
        load_scales<SPS>(ra, psa, STRIDE);
        half(I1{}, I0{}, rb.b0, rb.sc, o, o1);
        rb.b0 = ldg_stream_v4(plb + STRIDE);
        half(I1{}, I1{}, rb.b1, rb.sc, o, o1);
        rb.b1 = ldg_stream_v4(plb + STRIDE + 512);
        load_scales<SPS>(rb, psb, STRIDE);
        red_add_f32(accp, o);
        if constexpr (BT != 1) red_add_f32(accp + Mpad, o1);
        pla += STRIDE; psa += STRIDE; plb += STRIDE; psb += STRIDE; pp += STRIDE;
        accp += kWarps * 32;
    }
    {
        float o = 0.f, o1 = 0.f;
        half(I0{}, I0{}, ra.b0, ra.sc, o, o1);
        half(I0{}, I1{}, ra.b1, ra.sc, o, o1);
        half(I1{}, I0{}, rb.b0, rb.sc, o, o1);
        half(I1{}, I1{}, rb.b1, rb.sc, o, o1);
        red_add_f32(accp, o);
        if constexpr (BT != 1) red_add_f32(accp + Mpad, o1);
    }
}

// First L2 prefetches of a run of row blocks (issued before the tables are built): the first
// kPrefetchTrips blocks of D*kWarps items, one D-item request per lane.
__device__ __forceinline__ void prefetch_run_head(const uint8_t *pair_items, int item_bytes, int D, int kWarps, int rb_lo, int rb_hi,
                                                  int trips = kPrefetchTrips)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane < trips) {
        int rb = rb_lo + lane * D * kWarps + D * warp;
        int cnt = min(D, rb_hi - rb);
        if (cnt > 0) prefetch_l2(pair_items + (int64_t)rb * item_bytes, (uint32_t)(cnt * item_bytes));
    }
}

#ifdef FB_TRACE
// Instrumented build only: per-CTA phase timestamps (globaltimer, ns) of the last eight launches.
// Slots: 0 CTA start, 11 before / 1 after the wait for the predecessor, 3 end of the CTA's last layer;
// accumulated durations: 7 share and layer set-up, 9 input fetch (incl. the wait), 8 barrier before a build,
// 4 table build, 5 row loop, 10 tile counts, 6 reduction epilogue, 2 drawing a share.
__device__ unsigned long long g_fb_trace[8][1024][12];
__device__ __forceinline__ unsigned long long trace_now()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
#define FB_TRACE_ROW g_fb_trace[P.trace_slot & 7][blockIdx.x]
#define FB_TRACE_ON (threadIdx.x == 0 && blockIdx.x < 1024)
#define FB_TRACE_AT(slot) do { if (FB_TRACE_ON) FB_TRACE_ROW[slot] = trace_now(); } while (0)
#define FB_TRACE_T0(var) unsigned long long var = trace_now()
#define FB_TRACE_ADD(slot, var) do { if (FB_TRACE_ON) FB_TRACE_ROW[slot] += trace_now() - var; } while (0)
#define FB_TRACE_SET(var) var = trace_now()
#define FB_TRACE_ZERO() do { if (FB_TRACE_ON) { for (int i_ = 1; i_ < 12; ++i_) FB_TRACE_ROW[i_] = 0; } } while (0)
#else
#define FB_TRACE_AT(slot)
#define FB_TRACE_T0(var)
#define FB_TRACE_ADD(slot, var)
#define FB_TRACE_SET(var)
#define FB_TRACE_ZERO()
#endif

// Stage (iii) for the entry a CTA has just finished contributing to: publish, take a ticket per
// touched tile of rows; whoever arrives last at a tile converts it and re-zeroes the accumulator.
template <int BT>
__device__ __forceinline__ void reduce_and_store(const LinearEntry &E, int nb, int y_fp32, int *tile_cnt, int *done_list)
{
    const int tid = threadIdx.x;
    constexpr int kThreads = Cfg<BT>::kThreads;
    __threadfence();
    __syncthreads();
    const int npairs = E.arrivals;
    for (int t = tid; t < E.ntiles; t += kThreads) {
        int c = tile_cnt[t];
        int last = 0;
        if (c > 0) {
            int rbs = min(E.tile_rb, E.nrb - t * E.tile_rb);
            unsigned old = atomicAdd(E.tickets + t, (unsigned)c);
            last = (old + (unsigned)c == (unsigned)(npairs * rbs));
        }
        tile_cnt[t] = last;
    }
    __syncthreads();
    if (tid < 32) {                                // warp 0 compacts the completed tiles into a list, in place:
                                                   // a tile's slot in the list never lies beyond its own index
        int cnt = 0;
        for (int base = 0; base < E.ntiles; base += 32) {
            int t = base + tid;
            int f = (t < E.ntiles) ? tile_cnt[t] : 0;
            unsigned m = __ballot_sync(0xffffffffu, f);
            if (f) done_list[cnt + __popc(m & ((1u << tid) - 1u))] = t;
            cnt += __popc(m);
        }
        if (tid == 0) done_list[kMaxTiles] = cnt;
    }
    __syncthreads();
    const int ndone = done_list[kMaxTiles];
    if (ndone > 0) {
        __threadfence();
        // All rows of all completed tiles, in 4-row groups: every group is requested with one asynchronous 16-byte
        // copy from the accumulators (L2) into the table area, which is free by now -- no registers are held while
        // the copies fly, so one round trip serves every tile the CTA completed (up to 16K rows per batch) however
        // many there are -- then the groups are converted from shared memory and the accumulators re-zeroed.
        const int gpt = E.tile_rb * 8;                 // 4-row groups per tile
        constexpr int NV = nvec(BT);
        const int total = ndone * gpt * NV;
        // a gated pair stages the partner layer's groups behind its own (half the groups per batch)
        const int role = E.role();
        const int kStageGroups = role ? TabCfg<BT>::kTableBytes / 32 : TabCfg<BT>::kTableBytes / 16;
        // group idx of the flat list -> batch vector, first row, element offset in the accumulators (-1: padding rows)
        auto decode = [&](int idx, int &bb, int &row) -> int {
            const int li = idx / (gpt * NV), rem = idx - li * (gpt * NV);
            bb = rem / gpt;
            row = (done_list[li] * gpt + (rem - bb * gpt)) * 4;
            return row < E.mpad() ? bb * E.mpad() + row : -1;
        };
        const bool vec_ok = (E.ldy & 3) == 0;          // rows in groups of four stay 8 / 16-byte aligned in y
        for (int b0 = 0; b0 < total; b0 += kStageGroups) {
            const int n = min(kStageGroups, total - b0);
            for (int i = tid; i < n; i += kThreads) {
                int bb, row;
                const int eoff = decode(b0 + i, bb, row);
                if (eoff >= 0) {
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(kTabBase + 16u * (uint32_t)i),
                                 "l"(__cvta_generic_to_global(E.acc + eoff)) : "memory");
                    if (role)
                        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(kTabBase + 16u * (uint32_t)(kStageGroups + i)),
                                     "l"(__cvta_generic_to_global(E.acc2 + eoff)) : "memory");
                }
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            __syncthreads();
            for (int i = tid; i < n; i += kThreads) {
                int bb, row;
                const int eoff = decode(b0 + i, bb, row);
                if (eoff < 0) continue;
                float4 v;
                asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(kTabBase + 16u * (uint32_t)i));
                __stcg((float4 *)(E.acc + eoff), make_float4(0.f, 0.f, 0.f, 0.f));
                if (role) {
                    // SiLU-gated product of the two layers of the pair: y = silu(gate) * up, in fp32
                    float4 p;
                    asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(p.x), "=f"(p.y), "=f"(p.z), "=f"(p.w) : "r"(kTabBase + 16u * (uint32_t)(kStageGroups + i)));
                    __stcg((float4 *)(E.acc2 + eoff), make_float4(0.f, 0.f, 0.f, 0.f));
                    const float4 g = role == 1 ? v : p, u = role == 1 ? p : v;
                    v.x = g.x / (1.f + expf(-g.x)) * u.x;
                    v.y = g.y / (1.f + expf(-g.y)) * u.y;
                    v.z = g.z / (1.f + expf(-g.z)) * u.z;
                    v.w = g.w / (1.f + expf(-g.w)) * u.w;
                }
                if (bb >= nb) continue;
                if (vec_ok && row + 3 < E.M) {
                    if (y_fp32) {
                        *(float4 *)((float *)E.y + (int64_t)bb * E.ldy + row) = v;
                    } else {
                        const __half2 lo = __floats2half2_rn(v.x, v.y), hi = __floats2half2_rn(v.z, v.w);
                        uint2 pk;
                        pk.x = *(const uint32_t *)&lo;
                        pk.y = *(const uint32_t *)&hi;
                        *(uint2 *)((__half *)E.y + (int64_t)bb * E.ldy + row) = pk;
                    }
                    continue;
                }
                const float e[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    if (row + k >= E.M) break;
                    if (y_fp32) ((float *)E.y)[(int64_t)bb * E.ldy + row + k] = e[k];
                    else ((__half *)E.y)[(int64_t)bb * E.ldy + row + k] = __float2half_rn(e[k]);
                }
            }
            __syncthreads();       // the stage is reused by the next batch (and by the next table build)
        }
        for (int li = tid; li < ndone; li += kThreads) E.tickets[done_list[li]] = 0;
    }
    __syncthreads();       // done_list / tile_cnt are reused by the next entry
}

template <int SPS0, int SPS1, int BT, int NP>
__global__ void __launch_bounds__(Cfg<BT>::kThreads, Cfg<BT>::kMinBlocks)
fluxbin_linear_kernel(const __grid_constant__ LaunchParams P)
{
    constexpr int kThreads = Cfg<BT>::kThreads, kWarps = Cfg<BT>::kWarps;
    // dynamic shared memory: [kTabBase, +tables) at a fixed window address, small buffers after it
    extern __shared__ __align__(16) uint8_t smem[];
    const uint32_t smem_base = (uint32_t)__cvta_generic_to_shared(smem);
    if (smem_base > kTabBase) return;                                    // the host probes this first
    uint8_t *small = smem + (kTabBase - smem_base) + TabCfg<BT>::kTableBytes;
    float *abuf = (float *)small;
    int *tile_cnt = (int *)(abuf + TabCfg<BT>::kScratchFloats);
    int *done_list = tile_cnt;                     // compacted in place over the counters
    int *range = tile_cnt + kMaxTiles + 4;        // [2]: the share a CTA has drawn
    LinearEntry *Es = (LinearEntry *)(range + 8);  // the current entry, copied once (128 bytes)
    static_assert(sizeof(LinearEntry) == 128, "entry copy below moves 32 words");
    static_assert(NP == 1 || geom(BT) == 1, "two table sets side by side need 4-byte table entries");
    static_assert(BT == 1 || BT == 2 || BT == 4 || BT == 16 + 2 || BT == 16 + 4 || BT == 16 + 8 || BT == 32 + 1 || BT == 32 + 2 ||
                  BT == 32 + 4, "launch mode");
    static_assert(NP == 1 || !mu4(BT), "mu = 4 walks one pair per row block");
    const int tid = threadIdx.x;
    FB_TRACE_AT(0);
    FB_TRACE_ZERO();

    // Programmatic dependent launch: let the next kernel in the stream start its own prologue as soon
    // as SM resources free up; below, this kernel in turn waits for its predecessor only at the point
    // where it first touches data the predecessor may have written (activations, workspace) -- everything
    // that reads the packed layer alone (share bounds, column tables, the first weight bytes and the L2
    // prefetches behind them) runs ahead of that.
    asm volatile("griddepcontrol.launch_dependents;");
    bool predecessor_done = false;

    LaneAddr<BT> la;
    la.init(tid & 31);

    // The host has cut the cost line of the launch: the first gridDim.x shares are dealt one per CTA; any
    // further (small) shares are drawn from a counter by whichever CTA finishes first (no CTA waits for
    // another).  Co-resident CTAs do not progress at the same speed (the warp schedulers favour the older
    // ones), so the quick ones pick up the small shares and the SM stays fully occupied until the end.
    for (int share = blockIdx.x; share < P.nshares;) {
    FB_TRACE_T0(t_pro);
    int e0, i0, e1, i1;
    if (P.cuts) {
        const int2 c0 = __ldg((const int2 *)P.cuts + share), c1 = __ldg((const int2 *)P.cuts + share + 1);
        e0 = c0.x; i0 = c0.y; e1 = c1.x; i1 = c1.y;
    } else {
        e0 = 0; e1 = 0;
        i0 = P.single_cut[share];
        i1 = P.single_cut[share + 1];
    }

    for (int e = e0; e <= e1; ++e) {
        if (e == e1 && i1 == 0) break;             // the share ends where entry e1 begins (also: e1 == n)
        const LinearEntry *src = P.table ? P.table + e : &P.single;
        if (tid < 32) ((uint32_t *)Es)[tid] = ((const uint32_t *)src)[tid];
        __syncthreads();
        const LinearEntry &E = *Es;
        // With NP == 2 region 0 is walked two pairs at a time, their table sets side by side (4-byte entries,
        // every entry with an even number of global pairs): a "work pair" is then a couple of pairs, a
        // work row block their two items.
        // (NP is a kernel template parameter: the host picks the two-pair kernel when a CTA's share is worth
        // a couple of hundred items; below that building two table sets per run costs more than the better row
        // loop gains.  Deciding it at run time was measured slower than either variant: both row loops in
        // one kernel cost registers.)
        const int wp0 = E.npairs[0] / NP;
        const int I0 = wp0 * E.nrb, I1 = E.npairs[1] * E.nrb;
        // (the counters are next touched behind the barrier that precedes every table build)
        for (int t = tid; t < E.ntiles; t += kThreads) tile_cnt[t] = 0;
        int cur = (e == e0) ? i0 : 0;
        const int end = (e == e1) ? i1 : I0 + I1;
        FB_TRACE_ADD(7, t_pro);
        if (cur >= end) { __syncthreads(); FB_TRACE_SET(t_pro); continue; }

        // a segment = the CTA's row blocks of one work pair
        auto desc_of = [&](int region, int pair) {
            return E.packed + E.off_coldesc + (size_t)((region ? E.npairs[0] : 0) + pair) * FB_PAIR_DESC_BYTES;
        };
        auto fetch_x_for = [&](int region, int pair, BuildInput<BT> &in) {
            fetch_build_x<BT>(in, E.x, E.ldx, P.nb, region ? -1 : (2 * pair) / E.Kb * 128, (2 * pair + 1) / E.Kb * 128, E.N);
        };
        // With 16-byte entries one CTA owns the SM, so nothing covers the load latency of a build's inputs: the
        // inputs of the CTA's next pair are requested before the rows of the current one (+2 % at batch 8 with
        // fp16 entries; with two or three CTAs per SM the others cover it and the extra registers only cost).
        constexpr bool kNextInputsEarly = geom(BT) == 4;
        BuildInput<BT> bin_next;
        bool have_next = false;
        while (cur < end) {
            const int region = cur >= I0;
            const int local = region ? cur - I0 : cur;
            const int wpair = local / E.nrb, rb_lo = local - wpair * E.nrb;
            const int seg_end = min(end, cur - rb_lo + E.nrb);
            const int rb_hi = rb_lo + (seg_end - cur);
            const int np = region ? 1 : NP;                 // pairs walked together in this segment
            const int pair = wpair * np;
            const int ib_full = region ? ItemBytes<SPS1>::value : ItemBytes<SPS0>::value;
            // the last salient pair may be stored narrow: 8 or 16 steps per item instead of 32
            const int steps = (SPS1 == 1 && region && pair == E.npairs[1] - 1) ? E.sal_last_w() : 32;
            const int ib = steps == 32 ? ib_full : 96 * steps;
            const uint8_t *items = E.packed + E.off_items[region] + (size_t)pair * E.nrb * ib_full;
            const uint8_t *items_b = items + (size_t)E.nrb * ib_full;
            const int pf_d = np == 2 ? 1 : (region ? SPS1 : SPS0) == 1 ? 1 : DepthFor<BT>::value;
            // weights start moving now.  The two-pair loop prefetches the trip two ahead, so its head covers
            // trips 0 and 1 (+2 %); longer heads were measured slower in every launch mode.
            const int head_trips = np == 2 ? kPrefetchTrips + 1 : kPrefetchTrips;
            prefetch_run_head(items, ib, pf_d, kWarps, rb_lo, rb_hi, head_trips);
            if (np == 2) prefetch_run_head(items_b, ib, pf_d, kWarps, rb_lo, rb_hi, head_trips);

            FB_TRACE_T0(t_fetch);
            // (fetching the next pair's inputs ahead of the lookups was measured 15 % slower: the extra
            // live registers push the lookup loop over the 80-register budget of 3 CTAs per SM)
            BuildInput<BT> bin, bin_b;
            const bool reuse = kNextInputsEarly && have_next;
            if (!reuse) {
                fetch_build_desc<BT>(bin, desc_of(region, pair));
                if (np == 2) fetch_build_desc<BT>(bin_b, desc_of(region, pair + 1));
            }
            // region 0, one pair at a time (short runs): first item in flight during the build.  (With two
            // pairs per row block the runs are long and the extra live registers cost more than they hide.)
            ItemRegs<SPS0> pre;
            if (NP == 1 && region == 0) preload_first<SPS0, BT>(pre, items, rb_lo, rb_hi);

            if (!predecessor_done) {
                FB_TRACE_AT(11);
                asm volatile("griddepcontrol.wait;" ::: "memory");
                predecessor_done = true;
                FB_TRACE_AT(1);
            }
            if constexpr (kNextInputsEarly) {
                if (reuse) bin = bin_next; else fetch_x_for(region, pair, bin);
            } else {
                fetch_x_for(region, pair, bin);
                if (np == 2) fetch_x_for(region, pair + 1, bin_b);
            }
            FB_TRACE_T0(t_build);
            __syncthreads();     // previous segment's lookups are done before the tables are overwritten
            FB_TRACE_ADD(8, t_build);
            FB_TRACE_ADD(9, t_fetch);
            if (np == 2) {
                if constexpr (geom(BT) == 1) build_tables2<BT>(bin, bin_b, abuf);
            } else {
                build_tables<BT>(bin, abuf);
            }
            // the column tables of the next run's pairs (1 KB each, read once per run: otherwise an HBM miss on the
            // serial path of the next build) start moving into L2 now (+0.5 to 0.8 % in every launch mode)
            if (tid < 8 * np && pair + np < E.npairs[region])
                prefetch_line_if(desc_of(region, pair + np) + tid * 128, true);
            if constexpr (kNextInputsEarly) {
                // the CTA's next segment is the next pair of this entry's global region: its inputs start moving now
                have_next = seg_end < end && seg_end < I0;
                if (have_next) {
                    fetch_build_desc<BT>(bin_next, desc_of(0, pair + 1));
                    fetch_x_for(0, pair + 1, bin_next);
                }
            }
            FB_TRACE_ADD(4, t_build);
            FB_TRACE_T0(t_rows);
            if (region == 0) {
                if constexpr (NP == 2) process_rows2<SPS0, BT>(items, items_b, rb_lo, rb_hi, la, E.acc, E.mpad());
                else process_rows<SPS0, BT>(items, rb_lo, rb_hi, la, E.acc, E.mpad(), &pre);
            } else if (steps == 32) {
                process_rows<SPS1, BT>(items, rb_lo, rb_hi, la, E.acc, E.mpad());
            } else if constexpr (SPS1 == 1) {
                if (steps == 16) process_rows<1, BT, 16>(items, rb_lo, rb_hi, la, E.acc, E.mpad());
                else process_rows<1, BT, 8>(items, rb_lo, rb_hi, la, E.acc, E.mpad());
            }

            FB_TRACE_ADD(5, t_rows);
            FB_TRACE_T0(t_cnt);
            // how many items this CTA contributed to each tile of rows
            const int t_lo = rb_lo / E.tile_rb, t_hi = (rb_hi - 1) / E.tile_rb;
            for (int t = t_lo + tid; t <= t_hi; t += kThreads) {
                int a = max(rb_lo, t * E.tile_rb), b = min(rb_hi, (t + 1) * E.tile_rb);
                tile_cnt[t] += (b - a) * np;     // one thread per tile, segments are serial: no race
            }
            cur = seg_end;
            FB_TRACE_ADD(10, t_cnt);
        }
        FB_TRACE_T0(t_red);
        reduce_and_store<BT>(E, P.nb, P.y_fp32, tile_cnt, done_list);
        FB_TRACE_ADD(6, t_red);
        FB_TRACE_AT(3);
        FB_TRACE_SET(t_pro);
    }
        FB_TRACE_T0(t_draw);
        if (P.nshares <= (int)gridDim.x) break;    // one share per CTA: nothing to draw
        if (!predecessor_done) {
            asm volatile("griddepcontrol.wait;" ::: "memory");
            predecessor_done = true;
        }
        if (tid == 0) range[2] = (int)gridDim.x + (int)atomicAdd(P.counters, 1u);
        __syncthreads();
        share = range[2];
        __syncthreads();
        FB_TRACE_ADD(2, t_draw);
    }
    // the last CTA to leave puts the two launch counters back to zero for the next launch
    if (P.nshares > (int)gridDim.x && tid == 0) {
        unsigned old = atomicAdd(P.counters + 1, 1u);
        if (old == gridDim.x - 1) { P.counters[0] = 0u; P.counters[1] = 0u; }
    }
}

// Test hook: build one table set exactly as the kernel does and write it out as [32][256] fp32.
__global__ void __launch_bounds__(Cfg<1>::kThreads, 1)
fluxbin_debug_tables_kernel(const uint8_t *pair_desc, const uint16_t *x, float *out)
{
    constexpr int kThreads = Cfg<1>::kThreads;
    extern __shared__ __align__(16) uint8_t smem[];
    const uint32_t smem_base = (uint32_t)__cvta_generic_to_shared(smem);
    if (smem_base > kTabBase) return;
    uint8_t *tables = smem + (kTabBase - smem_base);
    BuildInput<1> bin;
    fetch_build_input<1>(bin, pair_desc, x, 0, 1, -1, -1, 0);
    build_tables<1>(bin, (float *)(tables + TabCfg<1>::kTableBytes));
    for (int i = threadIdx.x; i < 32 * 256; i += kThreads) {
        uint32_t sigma = i >> 8, p = i & 255;
        out[i] = *(const float *)(tables + (TabCfg<1>::lane_const(sigma) | (p << 8)));
    }
}

// Shared-window address at which dynamic shared memory starts for these kernels.
__global__ void fluxbin_smem_base_kernel(uint32_t *out)
{
    extern __shared__ __align__(16) uint8_t smem[];
    if (threadIdx.x == 0) *out = (uint32_t)__cvta_generic_to_shared(smem);
}

// dynamic shared memory to request: everything up to the end of the small buffers, as if the
// window began at 0 (the system-reserved bytes below the dynamic start are over-counted on purpose)
template <int BT> constexpr size_t smem_bytes() { return kTabBase + TabCfg<BT>::kTableBytes + TabCfg<BT>::kSmallBytes; }

} // namespace fbk
