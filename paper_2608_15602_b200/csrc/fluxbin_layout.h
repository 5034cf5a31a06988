// Private packed layout of one FluxBin layer (shared by the host packer and the kernels).
//
// Vocabulary
//   sub-vector   8 consecutive table columns (mu = 8); its 8 weight bits form one byte = one
//                table index (Eq. 15)
//   unit         16 sub-vectors that use one base: 128 input columns of a global base, or 16
//                salient sub-vectors of one salient base (virtual columns, Eq. 12)
//   pair         two units = 32 tables = one table set in shared memory
//   item         one pair x 32 output rows: 1024 bytes of weight bits + the row scales of those
//                rows, contiguous in memory; the unit of work of one warp iteration
//   region       0 = global bases, 1 = salient bases; a region has one `sps` (sub-vectors per
//                row-scale segment): 16 when a unit has one scale per row, 1 when every
//                sub-vector has its own
//
// Salient region with one scale per sub-vector (sps == 1): the salient sub-vectors of all bases form one flat
// list (base-major), cut into pairs of 32 with no padding in between; the last pair may hold only a few.  It
// is then stored NARROW, with w = 8 or 16 table slots instead of 32: its items carry w weight bytes and w
// scales per row (96 * w bytes), lane l walks steps 0 .. w-1 and still reads slot l ^ s -- the pair's column
// table repeats the w live tables 32 / w times, so slot l ^ s holds live table (l ^ s) mod w and the 32 lanes of
// a warp keep hitting 32 different banks.
//
// Item layout (lane l = row % 32 of the item; step s = 0..31):
//   at step s lane l uses table slot  sigma = l ^ s  (unit sigma>>4, sub-vector sigma&15), so the 32
//   lanes of a warp always address 32 different tables (different shared-memory banks).
//   bytes [h*512 + l*16 + c]           weight byte of step s = 16h + c                (h = 0,1)
//   bytes [1024 + ...]                 fp16 row scales, one per segment j = s / sps, lane-major
//                                      (for sps == 1: four 512-byte planes of 8 halves per lane)
// Narrow item (w = 8 or 16 steps):
//   bytes [l*w + s]                    weight byte of step s < w
//   bytes [32*w + ...]                 fp16 row scales of steps 0 .. w-1: w/8 planes of 8 halves per lane
#ifndef FLUXBIN_LAYOUT_H
#define FLUXBIN_LAYOUT_H

#include <stdint.h>

#define FB_MAGIC 0x31425846u /* "FXB1" */
#define FB_VERSION 3u
#define FB_HEADER_BYTES 256
#define FB_ROWS_PER_ITEM 32
#define FB_ITEM_BITS_BYTES 1024
#define FB_PAIR_DESC_BYTES 1024 /* 32 tables x 8 columns x {u16 x index, fp16 alpha} */

struct FbHeader {
    uint32_t magic, version;
    int32_t M, N, Kb, Ks, g, n_sal;
    int32_t Mpad, nrb;          // rows padded to 32; row blocks
    int32_t sps[2];             // sub-vectors per row-scale segment, per region
    int32_t nunits[2];
    int32_t npairs[2];
    int32_t item_bytes[2];
    int32_t n_sal_svec;         // salient sub-vectors per base after per-group padding
    int32_t n_dead;             // row-scale groups without any salient column
    int32_t sal_last_w;         // table slots of the last salient pair: 32, or 16 / 8 when it is stored narrow
    int32_t reserved0;
    uint64_t off_coldesc;       // [npairs0 + npairs1][32][8] {u16, u16}
    uint64_t off_items[2];      // region r: [npairs_r][nrb] items
    uint64_t off_sal_idx;       // int32 [n_sal]
    uint64_t off_dead_ids;      // int32 [n_dead]
    uint64_t off_dead_scales;   // u16 [Ks][n_dead][M]  (salient row scales no virtual column uses)
    uint64_t total_bytes;
    uint8_t reserved[FB_HEADER_BYTES - 4 * 2 - 4 * 20 - 8 * 7];
};

#ifdef __cplusplus
static_assert(sizeof(FbHeader) == FB_HEADER_BYTES, "header size");
#endif

#endif
