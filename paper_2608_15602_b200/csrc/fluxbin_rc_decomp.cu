// Row-column binary decomposition on the GPU (the step before packing): RC_Decomp of the paper's sub-routine
// listing (Algorithm 3) with the closed-form scale updates of Eq. 5 and the exhaustive sign search of Eq. 6,
// applied to every column group of g columns of a dense fp32 matrix on its own (the block loop of Algorithm 1
// without the Hessian compensation, which needs calibration data).  Output is the canonical layout
// fluxbin_pack takes: sign bits, fp16 row scales per (base, row, group), fp16 column scales per (base, column).
//
// All arithmetic is fp32.  The path is a sequence of memory-bound passes over W (no tensor cores: there is no
// contraction in it); one warp owns one (row, group) at a time, lane l the g/32 adjacent columns l*g/32 ... of
// the group, so a row of a group is one 128-bit load per lane and a lane's signs are adjacent bits of one word.
//
// Passes over W per call: 1 + T * K.  Every pass is local to a warp's (row, group) except the column form of
// Eq. 5, whose numerators are summed over all rows; so the steps are grouped into passes that end where that
// sum is needed:
//   first pass        greedy residual initialisation of all K bases, then the row form of Eq. 5 for base 1 and the
//                     numerators of its column form
//   per round, base k row form of Eq. 5 for base k (target = W - other bases) and the numerators of its column form
//   end of a round    the joint sign update of Eq. 6 (all 2^K tuples per element, lowest index on ties, one base at
//                     a time with single roundings) followed, in the same pass, by the next round's row form for
//                     base 1, which needs nothing but the new signs
//   column form       a_c(k) = numerator / (sum_i a_r^2 + eps): the numerators of a column group are reduced in
//                     shared memory over the 64 rows of a CTA, then one atomic per column and CTA; a small kernel
//                     behind the pass divides, stores and re-zeroes the accumulators.  (Folding that into the pass
//                     -- a ticket per group, the last CTA divides -- was measured slower: every CTA then ends with
//                     a fence and an atomic round trip, about 2 us of a 5 us CTA lifetime, 38 instead of ~30 us per
//                     pass at 4096 x 4096; CTAs that loop over several row blocks were slower still, 46 us.)
// Scales are stored as fp32 (working copy) and, rounded to nearest even, as fp16 whenever they are written.
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/fluxbin.h"
#include "fluxbin_internal.h"

namespace rcd {

constexpr int kWarpsPerCta = 8;
constexpr int kRowsPerWarp = 8;                       // a CTA covers 64 rows of one column group
constexpr int kRowsPerCta = kWarpsPerCta * kRowsPerWarp;
constexpr int kMaxK = 4;

struct Args {
    const float *W;        // [M][ldw]
    long long ldw;
    int M, N, g, NG, K;
    float eps;
    uint32_t *bits;        // [K][M][N/32]
    float *ar;             // [K][M][NG]
    float *ac;             // [K][N]
    uint16_t *ar16;        // the same, fp16 bit patterns
    uint16_t *ac16;
    const float *live;     // [N] 1 = real column, 0 = padding column (W must be 0 there); nullptr: all real
    float *colnum;         // [N]      numerators of the column form, zero between passes
    float *colden;         // [2][NG]  sum of a_r^2 per group, double buffered (see col_kernel)
};

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Column mapping: lane l owns the C = g / 32 ADJACENT columns l*C .. l*C + C-1 of the group, so its W values are one
// 128-bit load per row (C = 4), its signs are C adjacent bits of ONE sign word (word (l*C)/32 of the group, bit
// offset (l*C) % 32) and a sign word is assembled from 32/C neighbouring lanes with an OR over xor-shuffles.
template <int C> __device__ __forceinline__ void load_cols(float (&dst)[C], const float *p)
{
    if constexpr (C == 1) dst[0] = __ldg(p);
    else if constexpr (C == 2) { const float2 v = __ldg((const float2 *)p); dst[0] = v.x; dst[1] = v.y; }
    else {
#pragma unroll
        for (int c = 0; c < C; c += 4) {
            const float4 v = __ldg((const float4 *)(p + c));
            dst[c] = v.x; dst[c + 1] = v.y; dst[c + 2] = v.z; dst[c + 3] = v.w;
        }
    }
}

// OR of `v` over the aligned group of 32/C lanes that share a sign word; every lane of the group gets the word.
template <int C> __device__ __forceinline__ uint32_t gather_word(uint32_t v)
{
#pragma unroll
    for (int o = 1; o < 32 / C; o <<= 1) v |= __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Everything a warp needs from global memory for its kRowsPerWarp rows of one group, requested up front so that
// all of it is in flight at once (the passes are bound by load latency, not by arithmetic): the W values in
// registers, the sign words and row scales one or a few per lane, handed out by shuffles.
template <int C, int K> struct WarpRows {
    static constexpr int kWords = kRowsPerWarp * K * C;          // sign words [row][base][word of the group]
    static constexpr int kWordRegs = (kWords + 31) / 32;
    float w[kRowsPerWarp][C];
    uint32_t bw[kWordRegs];
    float arv;                                                   // row scale of (row, base) = lane, lane < 8 * K

    __device__ __forceinline__ void load_w(const Args &a, int G, int row0, int nrows, int lane)
    {
#pragma unroll
        for (int r = 0; r < kRowsPerWarp; ++r) {
            if (r < nrows) load_cols<C>(w[r], a.W + (long long)(row0 + r) * a.ldw + G * a.g + lane * C);
            else {
#pragma unroll
                for (int c = 0; c < C; ++c) w[r][c] = 0.f;
            }
        }
    }
    __device__ __forceinline__ void load_row_scales(const Args &a, int G, int row0, int nrows, int lane)
    {
        const int q = lane % K, r = lane / K;
        arv = (lane < kRowsPerWarp * K && r < nrows) ? a.ar[((size_t)q * a.M + row0 + r) * a.NG + G] : 0.f;
    }
    __device__ __forceinline__ void load_signs(const Args &a, int G, int row0, int nrows, int lane)
    {
        const int nw = a.N / 32;
#pragma unroll
        for (int m = 0; m < kWordRegs; ++m) {
            const int f = lane + 32 * m, c = f % C, q = (f / C) % K, r = f / (C * K);
            bw[m] = (f < kWords && r < nrows) ? a.bits[((size_t)q * a.M + row0 + r) * nw + G * C + c] : 0u;
        }
    }
    // the C sign bits of this lane's columns for (row r, base q), in the low bits; r, q compile-time after unrolling
    __device__ __forceinline__ uint32_t signs(int r, int q, int lane) const
    {
        const int f0 = (r * K + q) * C;                          // the group's C words never straddle a register
        const uint32_t word = __shfl_sync(0xffffffffu, bw[f0 >> 5], (f0 & 31) + (lane * C) / 32);
        return word >> ((lane * C) & 31);
    }
    __device__ __forceinline__ float ar(int r, int q) const { return __shfl_sync(0xffffffffu, arv, r * K + q); }
};

// the word index (within the group) this lane's columns live in, and whether this lane stores the gathered word
template <int C> __device__ __forceinline__ int word_of_lane(int lane) { return (lane * C) / 32; }
template <int C> __device__ __forceinline__ bool stores_word(int lane) { return (lane % (32 / C)) == 0; }

__device__ __forceinline__ uint16_t half_bits(float v) { return __half_as_ushort(__float2half_rn(v)); }

// v with its sign flipped when bit c of `bits` is set: a shift and one three-input logic operation, where a select
// between v and -v costs a bit test, a compare and the select (the passes are bound by issue slots).
__device__ __forceinline__ float flip_if_bit(float v, uint32_t bits, int c)       // c: compile-time after unrolling
{
    return __uint_as_float(__float_as_uint(v) ^ ((bits << (31 - c)) & 0x80000000u));
}

enum PassMode {
    kRow = 0,        // row form of Eq. 5 for base k (signs read from memory) + column numerators
    kSignRow = 1,    // Eq. 6 for all bases, then the row form for base 0 with the new signs + column numerators
    kSign = 2,       // Eq. 6 only (the last pass of a call)
    kInitRow = 3,    // greedy initialisation, then the row form for base 0 + column numerators
    kInit = 4        // greedy initialisation only (T == 0)
};

// (four CTAs per SM: 64 registers per thread hold a warp's eight rows without spills and 32 warps per SM cover the
// load latency better than 24 -- 4 % faster at 4096 x 4096, 6 % at 8192 x 8192; five CTAs per SM spill and lose 15 %;
// g = 256 holds twice the values per lane and keeps 128 registers)
template <int C, int K, int MODE> __global__ void __launch_bounds__(kWarpsPerCta * 32, C <= 4 ? 4 : 2) pass_kernel(Args a, int k_arg, int parity)
{
    constexpr bool kInitial = MODE == kInitRow || MODE == kInit;
    constexpr bool kSearch = MODE == kSignRow || MODE == kSign;
    constexpr bool kRowForm = MODE == kRow || MODE == kSignRow || MODE == kInitRow;
    __shared__ float part[kWarpsPerCta][C * 32];
    __shared__ float den_part[kWarpsPerCta];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int G = blockIdx.x, row0 = blockIdx.y * kRowsPerCta + warp * kRowsPerWarp;
    const int nw = a.N / 32;
    const int nrows = max(0, min(kRowsPerWarp, a.M - row0));
    const int k = MODE == kRow ? k_arg : 0;                // base of the row form

    // Programmatic dependent launch: the next kernel of the call may become resident while this one drains, and this
    // one requests its W values -- which no kernel of the call writes -- before it waits for its predecessor;
    // everything a predecessor wrote (signs, scales, zeroed accumulators) is read, and everything is written, after
    // the wait.  The first pass of a call waits first: whatever produced W may still be running.
    asm volatile("griddepcontrol.launch_dependents;");
    WarpRows<C, K> in;
    if constexpr (kInitial) asm volatile("griddepcontrol.wait;" ::: "memory");
    in.load_w(a, G, row0, nrows, lane);
    if constexpr (!kInitial) asm volatile("griddepcontrol.wait;" ::: "memory");
    if constexpr (MODE == kRow) in.load_signs(a, G, row0, nrows, lane);
    if constexpr (!kInitial) in.load_row_scales(a, G, row0, nrows, lane);
    float ack[K][C];                     // column scales of every base for this lane's columns
    float lv[C];                         // live mask (initial column scales)
    if constexpr (kInitial) {
        // initial column scales: 1 on real columns, 0 on padding columns (which then stay 0 through every update:
        // their numerators are sums of zeros); Eq. 5 with those scales divides by the number of real columns
#pragma unroll
        for (int c = 0; c < C; ++c) lv[c] = 1.f;
        if (a.live) load_cols<C>(lv, a.live + G * a.g + lane * C);
#pragma unroll
        for (int q = 0; q < K; ++q)
#pragma unroll
            for (int c = 0; c < C; ++c) ack[q][c] = lv[c];
    } else {
#pragma unroll
        for (int q = 0; q < K; ++q) load_cols<C>(ack[q], a.ac + (size_t)q * a.N + G * a.g + lane * C);
    }
    float akc[C];                        // those of base k
#pragma unroll
    for (int q = 0; q < K; ++q)
        if (q == k) {
#pragma unroll
            for (int c = 0; c < C; ++c) akc[c] = ack[q][c];
        }
    float den_c = 0.f;
#pragma unroll
    for (int c = 0; c < C; ++c) den_c += akc[c] * akc[c];
    den_c = warp_sum(den_c) + a.eps;                                      // sum_j (a_c B)^2 + eps, B^2 = 1
    const float inv_den = 1.f / den_c;                                   // (initial pass: 1 / (live columns + eps))
    float colsum[C];
#pragma unroll
    for (int c = 0; c < C; ++c) colsum[c] = 0.f;
    float ar2 = 0.f;
    float arn_mine = 0.f;                // lane r: the new row scale of row r

#pragma unroll
    for (int r = 0; r < kRowsPerWarp; ++r) {
        const int i = row0 + r;
        float arq[K];
        uint32_t sg[K];                  // the C sign bits of this lane's columns, per base
        if constexpr (kInitial) {
            float R[C];
#pragma unroll
            for (int c = 0; c < C; ++c) R[c] = in.w[r][c];
#pragma unroll
            for (int q = 0; q < K; ++q) {
                float s = 0.f;
#pragma unroll
                for (int c = 0; c < C; ++c) s += fabsf(R[c]) * lv[c];
                s = warp_sum(s) * inv_den;                                // Eq. 5 with a_c = 1 on the real columns
                uint32_t mine = 0u;
#pragma unroll
                for (int c = 0; c < C; ++c) {
                    const bool pos = R[c] >= 0.f;                         // sign(0) = +1
                    mine |= (pos ? 1u : 0u) << c;
                    const float step = s * lv[c];
                    R[c] = pos ? __fsub_rn(R[c], step) : __fadd_rn(R[c], step);
                }
                sg[q] = mine;
                arq[q] = s;
                if (lane == 0 && r < nrows && (MODE == kInit || q != 0)) {       // base 0's scale is replaced just below
                    a.ar[((size_t)q * a.M + i) * a.NG + G] = s;
                    a.ar16[((size_t)q * a.M + i) * a.NG + G] = half_bits(s);
                }
            }
        } else {
#pragma unroll
            for (int q = 0; q < K; ++q) arq[q] = in.ar(r, q);
            if constexpr (kSearch) {
#pragma unroll
                for (int q = 0; q < K; ++q) sg[q] = 0u;
#pragma unroll
                for (int c = 0; c < C; ++c) {
                    const float x = in.w[r][c];
                    float mag[K];
#pragma unroll
                    for (int q = 0; q < K; ++q) mag[q] = __fmul_rn(arq[q], ack[q][c]);        // rounded once
                    int best = 0;
                    float best_e = 0.f;
#pragma unroll
                    for (int t = 0; t < (1 << K); ++t) {
                        float e = x;
#pragma unroll
                        for (int q = 0; q < K; ++q) e = ((t >> q) & 1) ? __fsub_rn(e, mag[q]) : __fadd_rn(e, mag[q]);
                        e = fabsf(e);
                        if (t == 0 || e < best_e) { best_e = e; best = t; }                   // lowest index wins ties
                    }
#pragma unroll
                    for (int q = 0; q < K; ++q) sg[q] |= (uint32_t)((best >> q) & 1) << c;
                }
            } else {
#pragma unroll
                for (int q = 0; q < K; ++q) sg[q] = in.signs(r, q, lane);
            }
        }
        if constexpr (kInitial || kSearch) {
#pragma unroll
            for (int q = 0; q < K; ++q) {
                const uint32_t word = gather_word<C>((sg[q] & ((1u << C) - 1u)) << ((lane * C) & 31));
                if (stores_word<C>(lane) && r < nrows) a.bits[((size_t)q * a.M + i) * nw + G * C + word_of_lane<C>(lane)] = word;
            }
        }
        if constexpr (kRowForm) {
            // signs enter as a flip of the sign bit of one factor ((-a) * t and a * (-t) round alike, so which
            // factor carries the sign does not change a result)
            float t[C];
#pragma unroll
            for (int c = 0; c < C; ++c) t[c] = in.w[r][c];
#pragma unroll
            for (int q = 0; q < K; ++q) {
                if (q == k) continue;
#pragma unroll
                for (int c = 0; c < C; ++c)
                    t[c] = fmaf(flip_if_bit(arq[q], sg[q], c), ack[q][c], t[c]);      // what the other bases leave
            }
            uint32_t nsk = 0u;
#pragma unroll
            for (int q = 0; q < K; ++q) if (q == k) nsk = ~sg[q];
            float num = 0.f;
#pragma unroll
            for (int c = 0; c < C; ++c) {
                t[c] = flip_if_bit(t[c], nsk, c);                                      // B_k * target
                num = fmaf(akc[c], t[c], num);
            }
            const float arn = warp_sum(num) * inv_den;                                 // rows past M: W = 0 there, so 0
            if (lane == r) arn_mine = arn;
            ar2 = fmaf(arn, arn, ar2);
#pragma unroll
            for (int c = 0; c < C; ++c) colsum[c] = fmaf(arn, t[c], colsum[c]);
        }
    }
    if constexpr (kRowForm) {
        // lane r holds the new row scale of row r: one store per lane instead of eight by lane 0
        if (lane < nrows) {
            a.ar[((size_t)k * a.M + row0 + lane) * a.NG + G] = arn_mine;
            a.ar16[((size_t)k * a.M + row0 + lane) * a.NG + G] = half_bits(arn_mine);
        }
    }

    if constexpr (MODE == kInit) {
        // no update follows: the column scales are the initial ones
        if (blockIdx.y == 0 && warp == 0) {
#pragma unroll
            for (int q = 0; q < K; ++q)
#pragma unroll
                for (int c = 0; c < C; ++c) {
                    a.ac[(size_t)q * a.N + G * a.g + lane * C + c] = lv[c];
                    a.ac16[(size_t)q * a.N + G * a.g + lane * C + c] = half_bits(lv[c]);
                }
        }
    }
    if constexpr (kRowForm) {
#pragma unroll
        for (int c = 0; c < C; ++c) part[warp][lane * C + c] = colsum[c];
        if (lane == 0) den_part[warp] = ar2;
        __syncthreads();
        for (int j = threadIdx.x; j < C * 32; j += kWarpsPerCta * 32) {
            float s = 0.f;
#pragma unroll
            for (int w = 0; w < kWarpsPerCta; ++w) s += part[w][j];
            atomicAdd(a.colnum + G * a.g + j, s);
        }
        if (threadIdx.x == 0) {
            float s = 0.f;
            for (int w = 0; w < kWarpsPerCta; ++w) s += den_part[w];
            atomicAdd(a.colden + (size_t)(parity & 1) * a.NG + G, s);
        }
    }
}

// Column form of Eq. 5 behind a pass: a_c(k)_j = numerator_j / (sum_i a_r_i^2 + eps), fp32 and fp16; the accumulators go
// back to zero.  The group denominators are double buffered: this kernel reads buffer `parity` and clears the other
// one, which the next pass accumulates into -- no thread reads what another clears.  init_rest: the first pass
// of a call also gives the bases it did not update their initial column scales (the live mask).
__global__ void col_kernel(Args a, int k, int parity, int init_rest)
{
    asm volatile("griddepcontrol.launch_dependents;");
    asm volatile("griddepcontrol.wait;" ::: "memory");          // the pass before this has added all its numerators
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= a.N) return;
    const float v = a.colnum[j] / (a.colden[(size_t)(parity & 1) * a.NG + j / a.g] + a.eps);
    a.ac[(size_t)k * a.N + j] = v;
    a.ac16[(size_t)k * a.N + j] = half_bits(v);
    a.colnum[j] = 0.f;
    if (j < a.NG) a.colden[(size_t)((parity + 1) & 1) * a.NG + j] = 0.f;
    if (init_rest) {
        const float l = a.live ? a.live[j] : 1.f;
        for (int q = 0; q < a.K; ++q) {
            if (q == k) continue;
            a.ac[(size_t)q * a.N + j] = l;
            a.ac16[(size_t)q * a.N + j] = half_bits(l);
        }
    }
}

// launch with the programmatic-dependent-launch attribute (see pass_kernel)
template <typename... KArgs, typename... Args2>
static cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t s, Args2... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = 0;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

template <int C, int K> cudaError_t run(const Args &a, int T, cudaStream_t s)
{
    const dim3 grid(a.NG, (a.M + kRowsPerCta - 1) / kRowsPerCta), block(kWarpsPerCta * 32);
    const dim3 colgrid((unsigned)((a.N + 255) / 256)), colblock(256);
    cudaError_t e;
#define RCD_LAUNCH(...) do { e = launch_pdl(__VA_ARGS__); if (e != cudaSuccess) return e; } while (0)
    if (T == 0) {
        RCD_LAUNCH(pass_kernel<C, K, kInit>, grid, block, s, a, 0, 0);
        return cudaSuccess;
    }
    int parity = 0;
    RCD_LAUNCH(pass_kernel<C, K, kInitRow>, grid, block, s, a, 0, parity);
    RCD_LAUNCH(col_kernel, colgrid, colblock, s, a, 0, parity, 1);
    parity ^= 1;
    for (int it = 0; it < T; ++it) {
        for (int k = 1; k < a.K; ++k) {
            RCD_LAUNCH(pass_kernel<C, K, kRow>, grid, block, s, a, k, parity);
            RCD_LAUNCH(col_kernel, colgrid, colblock, s, a, k, parity, 0);
            parity ^= 1;
        }
        if (it + 1 < T) {
            RCD_LAUNCH(pass_kernel<C, K, kSignRow>, grid, block, s, a, 0, parity);
            RCD_LAUNCH(col_kernel, colgrid, colblock, s, a, 0, parity, 0);
            parity ^= 1;
        } else {
            RCD_LAUNCH(pass_kernel<C, K, kSign>, grid, block, s, a, 0, parity);
        }
    }
#undef RCD_LAUNCH
    return cudaSuccess;
}

} // namespace rcd

static size_t align256(size_t n) { return (n + 255) / 256 * 256; }
#define FB_CUDA(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) return fb::record_cuda_error((int)e_); } while (0)

extern "C" size_t fluxbin_rc_decomp_workspace_size(int32_t M, int32_t N, int32_t g, int32_t K)
{
    if (M < 1 || N < 32 || g < 32 || K < 1 || K > rcd::kMaxK || N % g != 0) return 0;
    const size_t NG = (size_t)N / g;
    return align256((size_t)K * M * NG * 4) + align256((size_t)K * N * 4) + align256((size_t)N * 4 + 2 * NG * 4);
}

extern "C" int32_t fluxbin_rc_decomp_passes(int32_t K, int32_t T)
{
    if (K < 1 || K > rcd::kMaxK || T < 0) return -1;
    return 1 + T * K;
}

extern "C" fluxbin_status_t fluxbin_rc_decomp(const float *d_W, int64_t ldw, const float *d_col_live, int32_t M, int32_t N,
                                              int32_t g, int32_t K,
                                              int32_t T, float eps, uint32_t *d_bits, uint16_t *d_row_scale,
                                              uint16_t *d_col_scale, float *d_row_scale_f32, float *d_col_scale_f32,
                                              void *d_workspace, size_t ws_bytes, void *cuda_stream)
{
    if (!d_W || !d_bits || !d_row_scale || !d_col_scale || !d_workspace) return FLUXBIN_ERR_NULL;
    if (M < 1 || N < 32 || N % 32 != 0 || g < 32 || g % 32 != 0 || N % g != 0 || ldw < N) return FLUXBIN_ERR_SHAPE;
    if (K < 1 || K > rcd::kMaxK || T < 0 || !(eps >= 0.f)) return FLUXBIN_ERR_RANGE;
    if (g != 32 && g != 64 && g != 128 && g != 256) return FLUXBIN_ERR_UNSUPPORTED;
    if (((uintptr_t)d_workspace & 15) != 0 || ((uintptr_t)d_W & 15) != 0 || (ldw & 3) != 0 || ((uintptr_t)d_col_live & 15) != 0 ||
        ((uintptr_t)d_col_scale_f32 & 15) != 0)
        return FLUXBIN_ERR_ALIGNMENT;
    if (ws_bytes < fluxbin_rc_decomp_workspace_size(M, N, g, K)) return FLUXBIN_ERR_BUFFER_TOO_SMALL;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    rcd::Args a;
    a.W = d_W; a.live = d_col_live; a.ldw = ldw; a.M = M; a.N = N; a.g = g; a.NG = N / g; a.K = K; a.eps = eps;
    a.bits = d_bits;
    a.ar16 = d_row_scale; a.ac16 = d_col_scale;
    uint8_t *ws = (uint8_t *)d_workspace;
    // the fp32 working copies of the scales live in the caller's fp32 outputs when those are given
    a.ar = d_row_scale_f32 ? d_row_scale_f32 : (float *)ws;     ws += align256((size_t)K * M * a.NG * 4);
    a.ac = d_col_scale_f32 ? d_col_scale_f32 : (float *)ws;     ws += align256((size_t)K * N * 4);
    a.colnum = (float *)ws;
    a.colden = a.colnum + N;
    FB_CUDA(cudaMemsetAsync(a.colnum, 0, (size_t)N * 4 + 2 * (size_t)a.NG * 4, s));
    cudaError_t e = cudaErrorInvalidValue;
#define RCD_K(CC) (K == 1 ? rcd::run<CC, 1>(a, T, s) : K == 2 ? rcd::run<CC, 2>(a, T, s) : K == 3 ? rcd::run<CC, 3>(a, T, s) : rcd::run<CC, 4>(a, T, s))
    switch (g / 32) {
    case 1: e = RCD_K(1); break;
    case 2: e = RCD_K(2); break;
    case 4: e = RCD_K(4); break;
    default: e = RCD_K(8); break;
    }
#undef RCD_K
    if (e != cudaSuccess) return fb::record_cuda_error((int)e);
    return FLUXBIN_OK;
}


// ---- the residual the salient refinement decomposes (Algorithm 2, step 3: R = W - W_g on the salient columns) ----
namespace rcd {
__global__ void salient_residual_kernel(const float *W, long long ldw, int M, int N, int g, int Kb, const uint32_t *bits,
                                        const float *ar, const float *ac, const int *sal_idx, const int *pos, int n_sal,
                                        float *P, long long ldp, float *live)
{
    const int v = blockIdx.x * blockDim.x + threadIdx.x, i = blockIdx.y;
    if (v >= n_sal) return;
    const int j = sal_idx[v], NG = N / g, nw = N / 32;
    float r = W[(long long)i * ldw + j];
    for (int k = 0; k < Kb; ++k) {
        const float m = __fmul_rn(ar[((size_t)k * M + i) * NG + j / g], ac[(size_t)k * N + j]);
        const bool plus = (bits[((size_t)k * M + i) * nw + j / 32] >> (j & 31)) & 1u;
        r = plus ? __fsub_rn(r, m) : __fadd_rn(r, m);
    }
    P[(long long)i * ldp + pos[v]] = r;
    if (i == 0) live[pos[v]] = 1.f;
}
} // namespace rcd

extern "C" fluxbin_status_t fluxbin_rc_salient_residual(const float *d_W, int64_t ldw, int32_t M, int32_t N, int32_t g, int32_t Kb,
                                                        const uint32_t *d_bits, const float *d_row_scale_f32,
                                                        const float *d_col_scale_f32, const int32_t *d_sal_idx,
                                                        const int32_t *d_pos, int32_t n_sal, float *d_P, int64_t ldp,
                                                        int32_t ncols_p, float *d_live, void *cuda_stream)
{
    if (!d_W || !d_bits || !d_row_scale_f32 || !d_col_scale_f32 || !d_sal_idx || !d_pos || !d_P || !d_live) return FLUXBIN_ERR_NULL;
    if (M < 1 || N < 32 || N % 32 != 0 || g < 32 || N % g != 0 || ldw < N || n_sal < 1 || ncols_p < 1 || ldp < ncols_p)
        return FLUXBIN_ERR_SHAPE;
    if (Kb < 1 || Kb > rcd::kMaxK || M > 65535) return FLUXBIN_ERR_RANGE;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    FB_CUDA(cudaMemset2DAsync(d_P, (size_t)ldp * 4, 0, (size_t)ncols_p * 4, M, s));
    FB_CUDA(cudaMemsetAsync(d_live, 0, (size_t)ncols_p * 4, s));
    const dim3 grid((n_sal + 127) / 128, M);
    rcd::salient_residual_kernel<<<grid, 128, 0, s>>>(d_W, ldw, M, N, g, Kb, d_bits, d_row_scale_f32, d_col_scale_f32, d_sal_idx,
                                                       d_pos, n_sal, d_P, ldp, d_live);
    FB_CUDA(cudaGetLastError());
    return FLUXBIN_OK;
}
