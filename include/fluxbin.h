/*
 * fluxbin.h -- C-ABI of the B200 (sm_100a) FluxBin decode linear layer.
 *
 * The layer computes  y = X * What^T  for a batch X of B activation vectors, where What is the
 * multi-binary-base weight of the paper (Def. 3.1 / Eq. 3 with one row scale per group of g
 * columns, plus the salient refinement of Eq. 9 on the columns listed in sal_idx):
 *
 *   What[i][j] = sum_{k<Kb} ar[k][i][j/g] * ac[k][j] * B[k][i][j]
 *              + sum_{k<Ks} [j = sal_idx[v]] * asr[k][i][j/g] * ascd[k][v] * Bsd[k][i][v]
 *
 * evaluated the LUT way (Sec. 3.2, Eq. 10-15): column scales are fused into the activations
 * (Eq. 11, Eq. 14), one table of 2^8 signed partial sums is built per 8-column sub-vector in
 * shared memory, packed weight bytes index the tables (Eq. 15), row scales are applied per
 * (row, group), and the salient columns are stored as dense "virtual columns" (VCM, Eq. 12-13)
 * so the salient branch runs through the same lookup loop.
 *
 * Conventions
 *   - M = output rows, N = input columns (the paper's M x N).
 *   - All scales and activations are IEEE fp16 bit patterns (uint16_t).  Arithmetic is fp32.
 *   - Bit 1 means +1, bit 0 means -1 (the 2b-1 of Eq. 14).
 *   - "host" / "device" is stated for every pointer.  The library never allocates device
 *     memory: packed weights, activations, outputs and workspace are owned by the caller.
 *   - Every entry point returns a status; none throws, aborts or prints.
 *   - Restrictions: N % 32 == 0, g % 32 == 0, N % g == 0, N <= 65536 (16-bit column index
 *     metadata, as in the paper's storage model), 1 <= Kb <= 4, 0 <= Ks <= 4, M >= 1.
 */
#ifndef FLUXBIN_H
#define FLUXBIN_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct fluxbin_weight fluxbin_weight_t; /* opaque host object describing one packed layer */

typedef enum {
    FLUXBIN_OK = 0,
    FLUXBIN_ERR_NULL = 1,             /* a required pointer is NULL */
    FLUXBIN_ERR_SHAPE = 2,            /* M/N/g violate the restrictions above */
    FLUXBIN_ERR_RANGE = 3,            /* Kb, Ks, B or a leading dimension out of range */
    FLUXBIN_ERR_SALIENT_MAP = 4,      /* sal_idx not strictly ascending or out of [0, N) */
    FLUXBIN_ERR_BUFFER_TOO_SMALL = 5, /* packed buffer or workspace smaller than required */
    FLUXBIN_ERR_ALIGNMENT = 6,        /* a device pointer is not 16-byte aligned */
    FLUXBIN_ERR_UNSUPPORTED = 7,      /* valid request this build cannot run (e.g. wrong GPU) */
    FLUXBIN_ERR_CUDA = 8,             /* a CUDA call failed; see fluxbin_last_cuda_error() */
    FLUXBIN_ERR_FORMAT = 9            /* packed buffer does not carry a valid header */
} fluxbin_status_t;

/*
 * One layer in canonical interchange layout (the problem statement of Sec. 3.2: parameter sets
 * Theta_k = {B, ar, ac}, Phi_k = {Bs, asr, asc} and the salient set I_sal).  All pointers are
 * HOST memory, borrowed for the duration of the call.
 */
typedef struct {
    int32_t M, N;      /* output rows, input columns */
    int32_t Kb, Ks;    /* global bases; extra bases on the salient columns (0 = no salient branch) */
    int32_t g;         /* columns per row-scale group; g == N gives one scale per row */
    int32_t n_sal;     /* number of salient columns, 0..N */
    const uint32_t *bits;          /* [Kb][M][N/32]; bit (j%32) of word j/32 set <=> B[k][i][j] = +1 */
    const uint16_t *row_scale;     /* [Kb][M][N/g] */
    const uint16_t *col_scale;     /* [Kb][N] */
    const int32_t  *sal_idx;       /* [n_sal] strictly ascending original column of virtual column v */
    const uint32_t *sal_bits;      /* [Ks][M][ceil(n_sal/32)] dense VCM matrix Bsd (Eq. 12): virtual
                                      column v is bit v%32 of word v/32; bits past n_sal must be 0 */
    const uint16_t *sal_row_scale; /* [Ks][M][N/g]; virtual column v uses group sal_idx[v]/g */
    const uint16_t *sal_col_scale; /* [Ks][n_sal] gathered column scale ascd (Eq. 13) */
} fluxbin_layer_desc_t;

/*
 * Bytes of the private packed representation of a layer (bit-packed bases in the kernel's tiled
 * order, row scales, fused column-scale/index table, salient map).  0 if the dimensions are
 * invalid.  Reads the dimension fields and, when it is non-NULL, sal_idx (the salient padding
 * depends on how the salient columns fall into row-scale groups); with sal_idx NULL the result
 * is an upper bound over all salient maps of that size.  The figure is the storage model of the
 * paper's appendix (S_base + S_sal) plus padding to the kernel's tiles.
 */
size_t fluxbin_packed_size(const fluxbin_layer_desc_t *desc);

/*
 * Validate a descriptor without packing it (dimension rules and the salient map).
 */
fluxbin_status_t fluxbin_validate(const fluxbin_layer_desc_t *desc);

/*
 * Pack into a HOST buffer of at least fluxbin_packed_size(desc) bytes (VCM, Def. 3.5: the
 * salient columns become dense virtual columns; bits are re-tiled for the lookup kernel).
 * Uses no GPU.  The result is position independent: copy it anywhere, then fluxbin_attach.
 */
fluxbin_status_t fluxbin_pack_host(const fluxbin_layer_desc_t *desc, void *h_packed, size_t bytes);

/*
 * Exact inverse of fluxbin_pack_host.  `out->M ... out->n_sal` are filled in; every non-NULL
 * array pointer of `out` must address caller-allocated HOST memory of the canonical size and is
 * written (the const qualifiers of the struct are ignored).  Bits, fp16 bit patterns and
 * indices round-trip bit-exactly.
 */
fluxbin_status_t fluxbin_unpack_host(const void *h_packed, size_t bytes, fluxbin_layer_desc_t *out);

/*
 * Read only the dimensions (M, N, Kb, Ks, g, n_sal) of a packed HOST buffer; pointers untouched.
 */
fluxbin_status_t fluxbin_packed_dims(const void *h_packed, size_t bytes, fluxbin_layer_desc_t *out);

/*
 * Pack `desc` and copy the result into the caller-owned DEVICE buffer d_packed (16-byte aligned,
 * d_bytes >= fluxbin_packed_size).  The copy is issued on `cuda_stream` (a cudaStream_t, NULL =
 * default stream) and the stream is synchronised before returning.  On success *out receives a
 * handle that borrows d_packed; release it with fluxbin_free (which never frees d_packed).
 */
fluxbin_status_t fluxbin_pack(const fluxbin_layer_desc_t *desc, void *d_packed, size_t d_bytes,
                              void *cuda_stream, fluxbin_weight_t **out);

/*
 * Make a handle for a DEVICE buffer that already holds a packed layer (e.g. after relocating
 * it).  `h_header` is HOST memory holding at least the first 256 bytes of that packed layer.
 */
fluxbin_status_t fluxbin_attach(const void *h_header, size_t header_bytes, void *d_packed, size_t d_bytes,
                                fluxbin_weight_t **out);

/*
 * Copy the packed layer back from the device and unpack it (see fluxbin_unpack_host).
 * Synchronises `cuda_stream`.
 */
fluxbin_status_t fluxbin_unpack(const fluxbin_weight_t *w, fluxbin_layer_desc_t *host_out, void *cuda_stream);

/* Dimensions of a handle (pointers of `out` untouched). */
fluxbin_status_t fluxbin_weight_dims(const fluxbin_weight_t *w, fluxbin_layer_desc_t *out);

/* CUDA device ordinal that was current when the handle was made, i.e. the device that holds d_packed; -1 on
 * NULL.  fluxbin_linear, fluxbin_linear_noalloc and fluxbin_plan_create / fluxbin_plan_run must be called with
 * that device current and return FLUXBIN_ERR_UNSUPPORTED otherwise (nothing is launched). */
int32_t fluxbin_weight_device(const fluxbin_weight_t *w);

/*
 * Precision of the lookup-table entries (Eq. 14) of batched launches (B >= 2) that read this layer.
 *
 *   FLUXBIN_TABLES_FP32 (default)  entries are fp32, the size the paper's shared-memory model counts
 *                                  (2^mu entries of 4 bytes per sub-vector and batch index); B runs in chunks
 *                                  of up to 4 vectors.
 *   FLUXBIN_TABLES_FP16            entries are the fp32 partial sums rounded once to fp16 (to nearest even),
 *                                  two batch vectors per 32-bit word: half the shared-memory bytes per lookup,
 *                                  which is what bounds the batched path; B runs in chunks of up to 8 vectors.
 *                                  Every sum is still accumulated in fp32.  Each lookup then carries a relative
 *                                  rounding error of at most 2^-11, so an output differs from the fp32-table
 *                                  result by about 2^-11 / sqrt(3) of the root-sum-square of its looked-up
 *                                  terms -- an error relative to the magnitude of the terms, not of the (possibly
 *                                  cancelling) sum.  Entries beyond the fp16 range (|sum of 8 fused activations|
 *                                  > 65504) become infinite and tiny ones lose bits below 6e-8: meant for
 *                                  normalised activations.
 *   FLUXBIN_TABLES_FP32_MU4        sub-vectors of mu = 4 columns instead of 8 (the paper's sub-vector-size study,
 *                                  "Impact of Sub-vector Size" and its table): every byte of weight bits indexes
 *                                  two 16-entry fp32 tables (Eq. 14 with mu = 4) instead of one 256-entry table, so
 *                                  the tables of 256 columns take 4 KB per batch vector instead of 32 KB and the
 *                                  lookups and their additions double.  The packed layer is the same; results agree with the
 *                                  mu = 8 path up to fp32 rounding order.  B runs in chunks of up to 4 vectors, and
 *                                  a single vector uses these tables too.  Only for layers whose row-scale groups
 *                                  are a multiple of 128 columns (FLUXBIN_ERR_UNSUPPORTED otherwise).
 *
 * With the first two formats a single vector (B == 1, or a trailing chunk of one) always uses fp32 entries of mu = 8.  The setting is read by
 * fluxbin_workspace_size, fluxbin_num_launches, fluxbin_linear and fluxbin_plan_create (all members of a plan
 * must agree, else FLUXBIN_ERR_UNSUPPORTED); change it only between those calls, and size workspaces after
 * it.  Returns FLUXBIN_ERR_RANGE for an unknown format.  fluxbin_get_table_format: the setting, -1 on NULL.
 */
#define FLUXBIN_TABLES_FP32 0
#define FLUXBIN_TABLES_FP16 1
#define FLUXBIN_TABLES_FP32_MU4 2
fluxbin_status_t fluxbin_set_table_format(fluxbin_weight_t *w, int32_t format);
int32_t fluxbin_get_table_format(const fluxbin_weight_t *w);

/*
 * DEVICE workspace bytes fluxbin_linear needs for batch size B with this layer: fp32 split-K
 * accumulators for one chunk of batch rows at a time plus one arrival counter per tile of output
 * rows (stage (iii) "reduction" of Sec. 3.2).  The workspace must be zeroed once with
 * fluxbin_workspace_init before its first use; every call leaves it zeroed again, so one
 * workspace of the maximum size can serve any sequence of stream-ordered calls.
 */
size_t fluxbin_workspace_size(const fluxbin_weight_t *w, int32_t B);

/* Zero a DEVICE workspace (asynchronous on cuda_stream). */
fluxbin_status_t fluxbin_workspace_init(void *d_workspace, size_t bytes, void *cuda_stream);

/*
 * y[b][i] = sum_j What[i][j] * x[b][j]   for b < B, i < M          (Eq. 10, computed per Eq. 11-15)
 *
 *   d_x   DEVICE fp16 [B][ldx], ldx >= N, 16-byte aligned base
 *   d_y   DEVICE [B][ldy], ldy >= M; fp32 if y_is_fp32 != 0 else fp16 (round-to-nearest-even of
 *         the fp32 result); every y[b][0..M) is overwritten
 *   d_workspace / ws_bytes   see fluxbin_workspace_size
 *
 * Asynchronous on cuda_stream; performs no allocation and no synchronisation, so calls can be
 * captured into a CUDA graph.  The kernel is launched with programmatic stream serialization: it may
 * begin (index arithmetic, L2 prefetch of its weights) while the previous kernel on the stream is
 * draining, and waits on the device before it reads d_x or touches the workspace.  B >= 1 arbitrary (processed in chunks of up to 4 vectors, 8 with fp16 table entries; a last chunk that would carry dead vectors in its table entries -- 3 vectors with fp32 entries, 5 or 6 with fp16 entries -- is cut into two launches when the layer, or the plan, holds at least 128 MiB of packed weights).  Calls
 * sharing a workspace must be ordered on one stream.  Accumulation is fp32 with fp32 atomics
 * across K slices, so results may differ in the last bits from run to run.
 */
fluxbin_status_t fluxbin_linear(const fluxbin_weight_t *w, const uint16_t *d_x, int32_t B, int64_t ldx,
                                void *d_y, int32_t y_is_fp32, int64_t ldy,
                                void *d_workspace, size_t ws_bytes, void *cuda_stream);

/*
 * fluxbin_linear for callers that may not allocate device memory.  (The paper has no counterpart:
 * this is a convenience of this library.)
 *
 * Who needs it: code that runs as a guest inside someone else's process -- an inference-server
 * backend, a plug-in, a callback on a latency-critical path -- and is handed its input and output
 * buffers but has no allocator of its own: the host application fixed the memory budget at start-up,
 * forbids cudaMalloc (it can synchronise the whole device and can fail once memory is fragmented),
 * and offers no per-call scratch.  Such a caller cannot provide the workspace fluxbin_linear asks for.
 *
 * Same arguments and result as fluxbin_linear, minus the workspace: the split-K accumulators and
 * arrival counters live in a fixed 1 MiB array inside the library image (fluxbin_noalloc_capacity();
 * every GPU that loads the library holds it until the process exits).  The call allocates nothing --
 * no cudaMalloc, no cudaFree, no allocating library routine.
 *
 *   - The rule: fluxbin_workspace_size(w, B) <= fluxbin_noalloc_capacity(), else FLUXBIN_ERR_BUFFER_TOO_SMALL.
 *     The workspace holds 4 bytes per output row (rounded up to 32 rows) for each accumulator row of a chunk of
 *     batch vectors, so 1 MiB takes about 260,000 output rows at B = 1, 130,000 at B = 2, 65,000 at B >= 3 with
 *     fp32 table entries (B = 3, 4 with fp16 entries) and 32,000 at B >= 5 with fp16 table entries.
 *   - The first call on each device looks up the device address of the array (with that device
 *     current) and keeps it; make that first call before any stream capture begins.  The current
 *     device must be the one that holds the layer, else FLUXBIN_ERR_UNSUPPORTED.
 *   - All calls on a device share the one array, which keeps the previous call's contents: each call
 *     clears the part it uses (cudaMemsetAsync on cuda_stream) before its kernel runs.  Two calls that
 *     overlap on the GPU (issued on different streams, or from several host threads at once) race
 *     on it and give wrong results; order them on one stream.
 */
fluxbin_status_t fluxbin_linear_noalloc(const fluxbin_weight_t *w, const uint16_t *d_x, int32_t B, int64_t ldx,
                                        void *d_y, int32_t y_is_fp32, int64_t ldy, void *cuda_stream);

/* Bytes of the fixed scratch array behind fluxbin_linear_noalloc. */
size_t fluxbin_noalloc_capacity(void);

/*
 * Test hook for the LUT identity (Eq. 14): build the tables of table-set `pair` (32 tables:
 * two runs of 16 consecutive 8-column sub-vectors) for activation row 0 of d_x exactly as the
 * kernel does, and write them as fp32 [32][256] to DEVICE d_tables.  h_cols (HOST, may be NULL)
 * receives the 32*8 source column indices and h_alpha the 32*8 fused column scales (fp16 bits)
 * the tables were built from, in table order.
 */
fluxbin_status_t fluxbin_debug_tables(const fluxbin_weight_t *w, const uint16_t *d_x, int32_t pair,
                                      float *d_tables, int32_t *h_cols, uint16_t *h_alpha, void *cuda_stream);

/*
 * Test hook for the work split (host only, uses no GPU): the bounds of the shares into which a launch of n packed
 * layers is cut.  The kernel walks the work items of a launch -- (pair or couple of pairs, block of 32 rows),
 * pair-major, layer after layer; the host cuts that list into `grid` shares of equal cost, one per CTA, plus
 * `nshares - grid` small ones drawn dynamically from the last (100 - static_percent) % of the cost.
 *
 *   h_headers            HOST array of n pointers, each to the first 256 bytes of a packed layer
 *   mode                 launch mode: 1, 2, 4 vectors with fp32 table entries, 16 + (2, 4, 8) with fp16 entries,
 *                        32 + (1, 2, 4) with fp32 entries of mu = 4 tables
 *   pairs_per_row_block  1 or 2 (2 needs an even number of global pairs in every layer)
 *   out_cuts             HOST int32 [nshares + 1][2]: {layer, work item} where share s begins; the last is {n, 0}
 *   out_work_items       HOST int32 [n] or NULL: work items of each layer
 */
fluxbin_status_t fluxbin_debug_cut_shares(int32_t n, const void *const *h_headers, int32_t mode, int32_t pairs_per_row_block,
                                          int32_t grid, int32_t nshares, int32_t static_percent, int32_t *out_cuts,
                                          int32_t *out_work_items);

/* Number of table sets (global + salient) of a layer; -1 on NULL. */
int32_t fluxbin_num_table_sets(const fluxbin_weight_t *w);

/* Kernel launches fluxbin_linear issues for this layer and batch size (for launch accounting): one per chunk of
 * batch vectors, see fluxbin_linear. */
int32_t fluxbin_num_launches(const fluxbin_weight_t *w, int32_t B);

/* Release the host object (never touches device memory).  NULL is allowed. */
void fluxbin_free(fluxbin_weight_t *w);

/*
 * A plan runs a fixed list of layers -- each with its own x and y -- in ONE persistent launch:
 * y_l = X_l * What_l^T for l < n (Eq. 10 for every layer).  The paper removes launch overhead from
 * its decode step by replaying all kernels from a CUDA graph (Experimental Setup); a plan goes one
 * step further and lets the table build and the split-K reduction of one layer overlap the weight
 * stream of the next.  Layers of a plan are independent: no member may read another member's
 * output (q/k/v or gate/up of a decoder layer qualify; so does any batch of unrelated layers).
 * Members may share an input.  All members must be of one row-scale format class -- g a multiple of
 * 128 with several groups per row; g == N (one scale per row) a multiple of 128; or one common
 * g < 128 -- otherwise FLUXBIN_ERR_UNSUPPORTED (members without salient columns only need to agree
 * on the class of their global bases).
 *
 *   w, d_x, ldx, d_y, ldy   HOST arrays of n handles / DEVICE pointers / leading dimensions
 *   d_table                 DEVICE buffer of fluxbin_plan_table_bytes(n, B) bytes, 16-byte aligned;
 *                           written here (stream synchronised) and read by every run
 *   d_workspace             DEVICE buffer of fluxbin_plan_workspace_bytes(...) bytes, zeroed once
 *                           with fluxbin_workspace_init before the first run; runs leave it zeroed
 * The pointers are captured at creation; all buffers must outlive the plan.
 */
typedef struct fluxbin_plan fluxbin_plan_t;

size_t fluxbin_plan_table_bytes(int32_t n, int32_t B);     /* enough for either table format */

size_t fluxbin_plan_workspace_bytes(int32_t n, const fluxbin_weight_t *const *w, int32_t B);

fluxbin_status_t fluxbin_plan_create(int32_t n, const fluxbin_weight_t *const *w,
                                     const uint16_t *const *d_x, const int64_t *ldx,
                                     void *const *d_y, const int64_t *ldy,
                                     int32_t B, int32_t y_is_fp32,
                                     void *d_table, size_t table_bytes,
                                     void *d_workspace, size_t ws_bytes,
                                     void *cuda_stream, fluxbin_plan_t **out);

/*
 * A plan with gated pairs: for each of the n_gated pairs {gate member, up member} in gate_up (HOST int32
 * [n_gated][2]) the plan writes  y = silu(What_gate x_gate) * (What_up x_up),  silu(t) = t / (1 + exp(-t)), into
 * the gate member's d_y instead of the two separate outputs (the gated feed-forward block of a decoder layer:
 * gate and up projections read the same input and only their product is needed).  The paper runs its linears as
 * separate kernels (Experimental Setup); here the CTA that completes a tile of rows of both layers converts both
 * accumulator tiles at once, so the two fp16 intermediates never reach memory.  Both sums are complete fp32
 * results of Eq. 10 when they are combined; the product is formed in fp32 and rounded once.
 * The two members of a pair must have the same number of rows (else FLUXBIN_ERR_SHAPE); a member belongs to at most
 * one pair and the indices must be valid (else FLUXBIN_ERR_RANGE); d_y / ldy of an up member are ignored (may be
 * NULL / 0).  Everything else as fluxbin_plan_create.
 */
fluxbin_status_t fluxbin_plan_create_gated(int32_t n, const fluxbin_weight_t *const *w,
                                           const uint16_t *const *d_x, const int64_t *ldx,
                                           void *const *d_y, const int64_t *ldy,
                                           const int32_t *gate_up, int32_t n_gated,
                                           int32_t B, int32_t y_is_fp32,
                                           void *d_table, size_t table_bytes,
                                           void *d_workspace, size_t ws_bytes,
                                           void *cuda_stream, fluxbin_plan_t **out);

/*
 * Launch the plan on cuda_stream: asynchronous, no allocation, no synchronisation (capturable).
 * Runs of plans that share a workspace must be ordered on one stream.
 */
fluxbin_status_t fluxbin_plan_run(const fluxbin_plan_t *plan, void *cuda_stream);

/* Kernel launches one fluxbin_plan_run issues (one per chunk of batch vectors, see fluxbin_linear); -1 on NULL. */
int32_t fluxbin_plan_num_launches(const fluxbin_plan_t *plan);

/* Introspection: how many table sets (pairs of 16-sub-vector units) the kernel of the plan's first launch keeps
 * resident per row block -- 2 when every member has an even number of global pairs, the table entries are 4 bytes
 * (batch 1, or batch 2 with fp16 entries) and each CTA's share of the plan is worth at least about 200 items (then
 * two pairs' row sums share one reduction, stage (iii)), else 1.
 * Both variants compute the same sums (Eq. 15) in a different order.  -1 on NULL. */
int32_t fluxbin_plan_pairs_per_row_block(const fluxbin_plan_t *plan);

/* Release the host object (never touches device memory).  NULL is allowed. */
void fluxbin_plan_free(fluxbin_plan_t *plan);

/* ---- the step before packing: row-column binary decomposition (Definition 3.1, Eq. 4-6, Algorithm 3) ----
 *
 * RC_Decomp of the paper's sub-routine listing on every column group of g columns of a dense matrix, each
 * group on its own (the block loop of Algorithm 1 without the Hessian error compensation, which needs
 * calibration data): greedy residual initialisation of the K bases, then T rounds of { for each base: row
 * scales by Eq. 5, column scales by Eq. 5 } followed by the joint sign update of Eq. 6 (all 2^K sign tuples per
 * element).  Readings where the paper is silent: the initial signs are sign(R) with sign(0) = +1, the initial
 * column scales 1 and the initial row scales Eq. 5 for those; with K >= 2 the target of base k's scale update is
 * W minus the other bases; ties of Eq. 6 go to the lowest tuple index sum_k [b_k = +1] 2^k.  A salient refinement
 * (mask) is run by handing over the gathered salient columns of the residual as the matrix.
 *
 *   d_W            device, fp32 [M][ldw] row-major, ldw >= N, 16-byte aligned with ldw % 4 == 0; read only
 *   d_col_live     device, fp32 [N], 16-byte aligned, or NULL: 1 for a real column, 0 for a padding column (a block
 *                  narrower than g -- the salient columns of a group -- is handed over padded with columns whose
 *                  W entries are 0; their column scales stay 0 and they do not enter Eq. 5).  NULL: all real.
 *   M, N, g        rows, columns, columns per group: N % g == 0, g in {32, 64, 128, 256}
 *   K, T, eps      bases 1..4, alternating rounds >= 0, the stability constant of Eq. 5 (>= 0)
 *   d_bits         device out, uint32 [K][M][N/32]: bit (j % 32) of word j/32 is 1 <=> B_ij = +1
 *   d_row_scale    device out, fp16 bit patterns [K][M][N/g]   } the canonical layout of a layer description,
 *   d_col_scale    device out, fp16 bit patterns [K][N]        } rounded to nearest even
 *   d_row_scale_f32, d_col_scale_f32   optional device out (NULL to skip): the same scales before rounding; when given
 *                  they serve as the working copies during the call (d_col_scale_f32 16-byte aligned)
 *   d_workspace    device scratch of fluxbin_rc_decomp_workspace_size() bytes, 16-byte aligned, any contents
 * All arithmetic is fp32.  Asynchronous on cuda_stream; allocates nothing; caller owns every buffer.
 * Errors: NULL / SHAPE / RANGE / UNSUPPORTED (other g) / ALIGNMENT / BUFFER_TOO_SMALL before any launch, CUDA.
 */
size_t fluxbin_rc_decomp_workspace_size(int32_t M, int32_t N, int32_t g, int32_t K);   /* 0 on invalid arguments */
/* Passes over W one call makes (each reads the fp32 matrix once): 1 + T * K -- the initialisation runs in the same
 * pass as the first row-scale update, and the sign update of a round in the same pass as the next round's first
 * row-scale update.  -1 on invalid arguments. */
int32_t fluxbin_rc_decomp_passes(int32_t K, int32_t T);
fluxbin_status_t fluxbin_rc_decomp(const float *d_W, int64_t ldw, const float *d_col_live, int32_t M, int32_t N, int32_t g,
                                   int32_t K, int32_t T, float eps, uint32_t *d_bits, uint16_t *d_row_scale, uint16_t *d_col_scale,
                                   float *d_row_scale_f32, float *d_col_scale_f32, void *d_workspace, size_t ws_bytes,
                                   void *cuda_stream);

const char *fluxbin_status_string(fluxbin_status_t s);

/* The cudaError_t of the most recent FLUXBIN_ERR_CUDA on the calling thread (0 if none). */
int fluxbin_last_cuda_error(void);

/*
 * The matrix the salient refinement decomposes (Algorithm 2, step 3): R = W - W_g restricted to the salient
 * columns, W_g the reconstruction from the global decomposition's outputs (fp32 scales and sign bits as
 * fluxbin_rc_decomp wrote them).  Virtual column v (input column d_sal_idx[v]) is written to column d_pos[v] of
 * the padded matrix d_P [M][ldp] (fp32, zero elsewhere: the call clears it first) and d_live [ncols_p] gets 1 at
 * d_pos[v], 0 elsewhere -- the pair of arguments fluxbin_rc_decomp takes for blocks narrower than its group.
 * All pointers device; M <= 65535; asynchronous on cuda_stream.  Errors: NULL / SHAPE / RANGE / CUDA.
 */
fluxbin_status_t fluxbin_rc_salient_residual(const float *d_W, int64_t ldw, int32_t M, int32_t N, int32_t g, int32_t Kb,
                                             const uint32_t *d_bits, const float *d_row_scale_f32,
                                             const float *d_col_scale_f32, const int32_t *d_sal_idx, const int32_t *d_pos,
                                             int32_t n_sal, float *d_P, int64_t ldp, int32_t ncols_p, float *d_live,
                                             void *cuda_stream);

/*
 * The canonical salient arrays from the outputs of the salient refinement (Algorithm 2, step 3).  The refinement
 * ran fluxbin_rc_decomp on the padded matrix fluxbin_rc_salient_residual wrote: one block of `width` columns per
 * row-scale group that holds salient columns (nblocks blocks; block b belongs to group d_block_group[b]; virtual
 * column v sits in column d_pos[v]).  This call gathers the sign bits of the virtual columns into the dense VCM
 * matrix (Eq. 12), scatters the blocks' row scales to their groups (zero for groups without salient columns) and
 * gathers the column scales (Eq. 13), rounding the scales to fp16 (to nearest even) on the device.
 *
 *   d_bits_p            device uint32 [Ks][M][width * nblocks / 32]   } as fluxbin_rc_decomp wrote them for the
 *   d_row_scale_p_f32   device fp32 [Ks][M][nblocks]                   } padded matrix (g = width)
 *   d_col_scale_p_f32   device fp32 [Ks][width * nblocks]              }
 *   d_pos, d_block_group   device int32 [n_sal], [nblocks]
 *   d_sal_bits          device out uint32 [Ks][M][ceil(n_sal / 32)]: bit v % 32 of word v / 32 = virtual column v
 *   d_sal_row_scale     device out fp16 bits [Ks][M][N / g];  d_sal_col_scale  device out fp16 bits [Ks][n_sal]
 *   d_sal_row_scale_f32, d_sal_col_scale_f32   optional device out (NULL to skip): the same before rounding
 * Asynchronous on cuda_stream; allocates nothing.  Errors: NULL / SHAPE / RANGE / CUDA.
 */
fluxbin_status_t fluxbin_rc_salient_collect(const uint32_t *d_bits_p, const float *d_row_scale_p_f32,
                                            const float *d_col_scale_p_f32, const int32_t *d_pos,
                                            const int32_t *d_block_group, int32_t M, int32_t N, int32_t g, int32_t Ks,
                                            int32_t n_sal, int32_t width, int32_t nblocks, uint32_t *d_sal_bits,
                                            uint16_t *d_sal_row_scale, uint16_t *d_sal_col_scale,
                                            float *d_sal_row_scale_f32, float *d_sal_col_scale_f32, void *cuda_stream);

/*
 * fluxbin_pack for canonical arrays that already live in DEVICE memory (the outputs of fluxbin_rc_decomp and
 * fluxbin_rc_salient_collect): the same packed bytes as fluxbin_pack_host (VCM, Def. 3.5), written by kernels, so
 * the arrays never cross host memory.
 *
 *   d_desc        HOST struct whose dimensions are as usual and whose array pointers are DEVICE memory in the
 *                 canonical layout (sal_idx included)
 *   h_sal_idx     HOST copy of the salient map [n_sal] (the header and the virtual-column structure are functions
 *                 of it); NULL when there is no salient branch
 *   d_packed      DEVICE buffer of at least fluxbin_packed_size bytes (computed with h_sal_idx), 16-byte aligned
 *   d_workspace   DEVICE scratch of fluxbin_pack_device_workspace_size(N, g, n_sal) bytes, 16-byte aligned
 * The stream is synchronised before returning.  On success *out receives a handle that borrows d_packed.
 * Errors: as fluxbin_pack.
 */
size_t fluxbin_pack_device_workspace_size(int32_t N, int32_t g, int32_t n_sal);     /* 0 on invalid arguments */
fluxbin_status_t fluxbin_pack_device(const fluxbin_layer_desc_t *d_desc, const int32_t *h_sal_idx, void *d_packed,
                                     size_t d_bytes, void *d_workspace, size_t ws_bytes, void *cuda_stream,
                                     fluxbin_weight_t **out);

#ifdef __cplusplus
}
#endif
#endif /* FLUXBIN_H */
