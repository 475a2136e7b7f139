/*
 * celty.h -- C ABI of the B200 (sm_100a) library for the batch-1 dual-sparse decode product
 *
 *     y = W . x      W: M x K, unstructured-pruned FP16, stored in 4-bit run-length coded CSC
 *                    x: K FP16 activations, made sparse at run time by magnitude thresholding
 *                    y: M FP32
 *
 * (Celty: sparse format Section 3.2, kernel formulation Section 3.1, index reconstruction
 * Algorithm 1, shared-memory scatter-accumulation Section 3.3.)
 *
 * Conventions
 *   - Every function returns 0 (CELTY_OK) or a negative celty_status; nothing throws or aborts.
 *   - "host" pointers are ordinary CPU memory, "device" pointers are CUDA device memory of the
 *     current device.  The library never allocates device memory: the caller provides it
 *     (celty_device_bytes says how much) and keeps it alive while the handle uses it.
 *   - celty_stream_t is a cudaStream_t passed as void* (NULL = the default stream).  Calls that
 *     take a stream only enqueue work on it and return without synchronising unless stated.
 *   - M = rows = outputs, K = columns = inputs.  W and mask are row-major on the host.
 *   - One handle must not be used from two streams or two threads at the same time: the
 *     compacted activation list and the status word live in the handle's workspace.
 */
#ifndef CELTY_H
#define CELTY_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct celty_matrix celty_matrix;   /* opaque: host copy of the encoded matrix + device binding */
typedef void *celty_stream_t;               /* cudaStream_t */

typedef enum {
    CELTY_OK = 0,
    CELTY_EINVAL = -1,     /* null pointer, size out of range, misaligned vector, bad option, tau < 0 or not finite */
    CELTY_ENOMEM = -2,     /* host allocation failed, or a caller-provided device buffer is too small */
    CELTY_ECUDA = -3,      /* a CUDA runtime call failed; celty_last_cuda_error() returns its code */
    CELTY_ESTATE = -4,     /* handle not bound to device memory yet */
    CELTY_ETIMEOUT = -5,   /* device status word: a bounded wait inside a kernel ran out */
    CELTY_EBOUNDS = -6,    /* device status word: a decoded row or list index was out of range */
    CELTY_ELIMIT = -7      /* a size exceeds the fixed scratch of celty_spmspv_static */
} celty_status;

/* Device-image layouts.  Both hold exactly the (value, 4-bit run) entries that Section 3.2
 * defines, one run per value; they differ in how entries are grouped for the kernel.
 *   CELTY_LAYOUT_COLUMN     tile_rows must be 0: runs are counted along the whole column.
 *                           A warp decodes 256 consecutive entries at a time with the intra-warp
 *                           prefix sum of Algorithm 1 and scatters with shared-memory atomics.
 *   CELTY_LAYOUT_LANE_TILE  tile_rows = R > 0: the rows are partitioned into tiles of R rows (the
 *                           row partition of Section 3.1 taken down to one tile per lane) and the
 *                           rule of Section 3.2 is applied to every tile separately.  Lane L of the
 *                           warp that works on slab s owns tile 32*s + L, so every lane writes its
 *                           own shared-memory bank: no conflicts, no atomics.  A tile is not a block
 *                           of consecutive rows: rows are dealt out like cards, row r to lane r mod 32
 *                           and every group of 32 rows, C groups at a time, to the S slabs in turn
 *                           (celty_row_map gives S, R and C):
 *                               row(s, L, i) = (((i / C) * S + s) * C + i mod C) * 32 + L
 *                           is local row i (0 <= i < R) of tile 32*s + L; values >= M do not exist.
 *                           Within a tile the rows grow with i, and "dropped rows since the previous
 *                           entry" counts local rows.  Every lane and every slab thus samples the
 *                           whole height of the matrix, whatever the row-wise density profile.
 */
enum { CELTY_LAYOUT_COLUMN = 0, CELTY_LAYOUT_LANE_TILE = 1 };

typedef struct {
    int32_t run_bits;    /* must be 4, the run width Section 3.2 settles on (Figure 3)               */
    int32_t layout;      /* CELTY_LAYOUT_COLUMN or CELTY_LAYOUT_LANE_TILE                             */
    int32_t tile_rows;   /* COLUMN: must be 0.  LANE_TILE: local rows per tile, 1..240, or 0 = choose */
    int32_t slabs_per_block; /* LANE_TILE: slabs of rows one thread block works on, 1..15; 0 = choose (1);
                                COLUMN: must be 0                                                         */
} celty_encode_opts;

/*
 * celty_encode -- offline packing of a pruned weight matrix into RLC-CSC (Section 3.2, Fig. 2(a)).
 *   W_host     M x K FP16 bit patterns, row-major, leading dimension ldw (elements, >= K).
 *   mask_host  M x K bytes, row-major, leading dimension K; non-zero = the weight is kept.
 *              NULL keeps every weight whose value is not +-0.
 *   opts       NULL = { 4, CELTY_LAYOUT_LANE_TILE, 0, 0 }.
 *   out        receives a new handle (free it with celty_destroy).
 * Per column (per row tile), rows ascending: every kept weight becomes one entry (value, run) with
 * run = number of dropped rows since the previous entry; a gap larger than 15 first emits
 * zero-valued padding entries (run 15, each standing for 15 dropped rows plus its own row).
 * Nothing is emitted after the last kept row.  The caller keeps ownership of W_host and mask_host;
 * the handle copies what it needs.  Limits: 1 <= M <= 49152 (one thread block's FP32 accumulators
 * must fit shared memory), 1 <= K < 2^31, at most 2^32 - 1 stored entries, at most 1024 tiles.
 * Errors: CELTY_EINVAL, CELTY_ENOMEM.
 */
int celty_encode(const uint16_t *W_host, int64_t ldw, const uint8_t *mask_host, int64_t M, int64_t K,
                 const celty_encode_opts *opts, celty_matrix **out);

/* Frees the handle and its host memory.  Device buffers stay with the caller.  NULL is allowed. */
void celty_destroy(celty_matrix *m);

/*
 * celty_clone -- a second handle holding a copy of the encoded matrix (host memory only; the copy is not
 * bound to device memory and has the library's default launch settings), for callers that want the same
 * layer resident several times (one binding per handle) without packing it again.
 * Errors: CELTY_EINVAL, CELTY_ENOMEM.
 */
int celty_clone(const celty_matrix *m, celty_matrix **out);

/*
 * celty_info -- sizes of the encoded matrix.  Any output pointer may be NULL.
 *   nnz               kept weights;  n_pad: padding entries;  stored entries = nnz + n_pad
 *   compressed_bytes  2.5 bytes per stored entry + 4 bytes per column pointer: the figure the
 *                     "compression efficiency" of Section 3.2 is the ratio of, over 2*M*K
 *   tile_rows, layout the values in effect (after "0 = choose")
 */
int celty_info(const celty_matrix *m, int64_t *M, int64_t *K, int64_t *nnz, int64_t *n_pad,
               int64_t *compressed_bytes, int32_t *layout, int32_t *tile_rows);

/*
 * celty_row_map -- the parameters of the LANE_TILE row map (see CELTY_LAYOUT_LANE_TILE): slabs S of
 * 32 tiles, local rows per tile R, chunk C.  The paper partitions rows into contiguous tiles
 * (Section 3.1); this library's tiles are the interleaved row sets given above.  For a COLUMN handle
 * the answer is S = 1, R = M, C = 1 (the single tile is the column).  Output pointers may be NULL.
 */
int celty_row_map(const celty_matrix *m, int32_t *slabs, int32_t *tile_rows, int32_t *chunk);

/*
 * celty_decode_host -- the stored entries of column `col`, decoded on the host from the handle's
 * own packed image (round-trip tests): absolute row (Algorithm 1: prefix sum of runs + ordinal),
 * FP16 bit pattern, run and pad flag of each entry, row tiles concatenated in ascending tile order
 * (LANE_TILE: tile 32*s + L, its entries by ascending local row).
 * cap = capacity of the output arrays (entries); *n receives the entry count even when it exceeds
 * cap (then nothing is written and CELTY_ENOMEM is returned).  Output pointers may be NULL.
 */
int celty_decode_host(const celty_matrix *m, int64_t col, int32_t *rows, uint16_t *vals, uint8_t *runs,
                      uint8_t *is_pad, int64_t cap, int64_t *n);

/*
 * celty_host_image -- read-only view of the packed image held by the handle (what
 * celty_bind_device copies to the device): pointer, size, and the offset at which the entry
 * stream starts (column metadata comes first).  Valid until celty_destroy.  The runs of 8
 * consecutive entries of a lane share one little-endian 32-bit word, entry e in bits 4e..4e+3.
 */
int celty_host_image(const celty_matrix *m, const void **image, size_t *image_bytes, size_t *stream_offset);

/*
 * celty_device_bytes -- how much device memory the caller must provide:
 *   image_bytes      the packed matrix as the kernels read it (column metadata + entry stream)
 *   workspace_bytes  per-handle scratch: compacted activation list (indices, values, count), the
 *                    status word, and the per-block partial sums of the split-K merge
 * Both are multiples of 256; the buffers must be 256-byte aligned.
 */
int celty_device_bytes(const celty_matrix *m, size_t *image_bytes, size_t *workspace_bytes);

/*
 * celty_bind_device -- attach caller-owned device memory and enqueue the host-to-device copy of
 * the image (and the clearing of the workspace) on `stream`.  The host image is ordinary pageable
 * memory, so the copy may block the calling thread; the handle is usable on `stream` on return
 * and on other streams after the caller has synchronised.
 * Errors: CELTY_EINVAL, CELTY_ENOMEM (buffer too small or misaligned), CELTY_ECUDA.
 */
int celty_bind_device(celty_matrix *m, void *image_dev, size_t image_bytes, void *workspace_dev,
                      size_t workspace_bytes, celty_stream_t stream);

/*
 * celty_compact -- activation compaction alone (magnitude thresholding, Sections 1 and 2.1; the
 * column skip of Section 3.1 made explicit):  S = { j : not(|x_j| <= tau) } in ascending j,
 * compared in FP32 after exact widening (tau = 0 drops exactly +-0; NaN survives).
 *   x_dev      K FP16 values (device, 16-byte aligned), not modified
 *   idx_dev    int32[K]   receives the surviving column indices   (device)
 *   val_dev    uint16[K]  receives their FP16 bit patterns        (device)
 *   count_dev  int32[1]   receives |S|                            (device)
 * Errors: CELTY_EINVAL (null, K <= 0, tau < 0 or not finite), CELTY_ECUDA.
 */
int celty_compact(const void *x_dev, int64_t K, float tau, int32_t *idx_dev, uint16_t *val_dev,
                  int32_t *count_dev, celty_stream_t stream);

/*
 * celty_spmspv -- the hot path: y = W . threshold(x, tau), batch 1 (Sections 3.1-3.3).
 * Enqueues on `stream` one kernel (LANE_TILE layout) that thresholds and compacts x, visits only
 * the surviving columns, decodes their runs to rows, accumulates value * x_j in shared memory in
 * FP32 (one rounding per multiply-add) and merges the thread blocks' results into y (FP32 adds in L2
 * by bulk reduce-add copies; celty_set_launch can select a sum in a fixed order instead); the COLUMN
 * layout uses a compaction kernel followed by the SpMSpV kernel.  On a stream of calls the kernel's
 * set-up overlaps the end of the previous kernel (programmatic dependent launch); it waits for that
 * kernel before it reads x or touches y or the workspace.
 *   x_dev  K FP16 (device, 16-byte aligned), not modified
 *   y_dev  M FP32 (device, 16-byte aligned), overwritten
 * The order of FP32 additions is not fixed (Section 4.2: scatter-accumulation is order-
 * independent), so results may differ in the last bits between calls.  Activations must be finite
 * for the result to equal the definition in every row: a zero-valued stored slot (a padding entry,
 * or a slot that fills a lane's last group of 8) times an infinite or NaN x_j is NaN.
 * Errors: CELTY_EINVAL, CELTY_ESTATE, CELTY_ECUDA.  A bounded wait that runs out inside the kernel does
 * not hang or fault: it sets the status word (CELTY_ETIMEOUT from celty_last_status).  Decoded row indices
 * are range-checked by the COLUMN kernel only (CELTY_EBOUNDS); the LANE_TILE kernels trust the image that
 * celty_encode built.
 */
int celty_spmspv(celty_matrix *m, const void *x_dev, float tau, void *y_dev, celty_stream_t stream);

/*
 * Work on y after the merge, inside the same launch (LANE_TILE handles, single-launch kernel, bulk reduce-add
 * merge).  Section 6.2 times the seven products of a decode layer; between the gate/up and the down projection of
 * its MLP sits SiLU(gate) * up, and every product's output feeds FP16 consumers.
 *   CELTY_EPILOGUE_FP16    out_fp16[i] = y[i] rounded to FP16 (nearest even), i < M; y keeps the FP32 values.
 *   CELTY_EPILOGUE_SWIGLU  the handle holds the gate projection's rows stacked on the up projection's
 *                          (M = 2I rows): h_i = SiLU(y_i) * y_{I+i} for i < I, evaluated in FP32, rounded once to
 *                          FP16 and stored in out_fp16[i]; every i with not(|h_i| <= tau) (the comparator of
 *                          celty_compact, applied to the rounded value) is appended to the list
 *                          (list_idx, list_val, list_count[0]), which celty_spmspv_list takes as the survivors of
 *                          the down projection.  The list comes out in no particular order (thread blocks append
 *                          to it as they finish); as a set it is exactly the thresholded h.  list_idx and list_val
 *                          need room for I entries.
 * All pointers are device memory of the current device.
 */
enum { CELTY_EPILOGUE_NONE = 0, CELTY_EPILOGUE_FP16 = 1, CELTY_EPILOGUE_SWIGLU = 2 };

typedef struct {
    int32_t kind;         /* CELTY_EPILOGUE_*                                              */
    void *out_fp16;       /* FP16: M values; SWIGLU: M / 2 values                          */
    float tau;            /* SWIGLU: threshold of the emitted list (finite, >= 0)          */
    int32_t *list_idx;    /* SWIGLU: int32[M / 2]                                          */
    uint16_t *list_val;   /* SWIGLU: FP16 bit patterns [M / 2]                             */
    int32_t *list_count;  /* SWIGLU: int32[1], overwritten                                 */
} celty_epilogue;

/*
 * celty_spmspv_ex -- celty_spmspv followed, in the same launch, by the work `ep` describes (NULL = none).
 * Errors: those of celty_spmspv; CELTY_EINVAL also for a COLUMN handle, the two-launch or the ordered-merge
 * variant, a missing output pointer, an odd M with SWIGLU.
 */
int celty_spmspv_ex(celty_matrix *m, const void *x_dev, float tau, void *y_dev, const celty_epilogue *ep,
                    celty_stream_t stream);

/*
 * celty_spmspv_list -- the same product when the thresholding (step a1) has already been done by whoever produced
 * the activations: y = sum over the n = count_dev[0] listed columns idx_dev[r] of column idx_dev[r] times the FP16
 * value val_dev[r].  The list may be in any order; every column at most once; n <= K.  This is how the down
 * projection consumes the list that CELTY_EPILOGUE_SWIGLU emits (the call reads the count on the device, so the
 * two calls can follow each other on a stream without a host round trip).  `ep` as in celty_spmspv_ex.
 * celty_last_compaction is not updated by this call (the count it reports is n).
 * Errors: CELTY_EINVAL, CELTY_ESTATE, CELTY_ECUDA.
 */
int celty_spmspv_list(celty_matrix *m, const int32_t *idx_dev, const uint16_t *val_dev, const int32_t *count_dev,
                      void *y_dev, const celty_epilogue *ep, celty_stream_t stream);

/*
 * celty_spmspv_batch -- the product for a small batch of N = 1 .. 8 activation vectors against the same matrix
 * (LANE_TILE handles):  y[n] = W . threshold(x[n], tau)  for every n.  Sections 2.2-2.3 place the method against
 * SpMM kernels that need N >= 8.  Two ways are built.  The widened scheme: a column is fetched once when any of the
 * N activations in it survives (the union of the surviving columns), and every stored entry is multiplied into N
 * accumulators; two launches (union compaction, product with plain loads and an atomic merge); taken when the
 * handle runs the two-launch variant (celty_set_launch, variant 1), has no workspace bound, or a row of x or y
 * does not start on a 16-byte boundary.  Otherwise N launches of the single-vector kernel, which measured faster at
 * every N (the widened kernels have room for fewer warps, and the union is nearly every column from N = 4 on);
 * celty_last_compaction then reports the last vector's list.
 *   x_dev  N rows of K FP16 values, row n at x_dev + n * ldx (elements), not modified
 *   y_dev  N rows of M FP32 values, row n at y_dev + n * ldy, overwritten
 *   list_scratch_dev  device scratch, 256-byte aligned, at least 256 + round_up(4 K, 256) + 16 K bytes (union list
 *                     and the N values of every listed column)
 * Errors: CELTY_EINVAL, CELTY_ESTATE, CELTY_ENOMEM (scratch too small or misaligned), CELTY_ELIMIT (the N
 * accumulators of one slab of rows do not fit shared memory), CELTY_ECUDA.
 */
int celty_spmspv_batch(celty_matrix *m, const void *x_dev, int64_t ldx, int32_t N, float tau, void *y_dev, int64_t ldy,
                       void *list_scratch_dev, size_t scratch_bytes, celty_stream_t stream);

/*
 * celty_shard_columns -- the column range [k_begin, k_end) of rank `rank` of `world` when a layer is sharded by
 * columns over several GPUs (each GPU encodes its own columns whole, thresholds its own slice of x and produces
 * a partial y; one all-reduce of M FP32 values then gives y -- the exchange is the caller's, e.g. NCCL through
 * torch.distributed).  The ranges tile [0, K) in rank order and start on multiples of 8 columns, so that a
 * shard's slice of x is 16-byte aligned.  Host-only.  Errors: CELTY_EINVAL.
 */
int celty_shard_columns(int64_t K, int32_t world, int32_t rank, int64_t *k_begin, int64_t *k_end);

/*
 * celty_spmspv_swiglu -- the down projection of an MLP whose activations are made inside the call: the input is the
 * FP32 result of the stacked [gate; up] product (gate_up_dev: 2K values, the K gate results first), and step a1
 * works on  x_j = SiLU(gate_j) * up_j  evaluated in FP32 and rounded once to FP16 -- the same values
 * CELTY_EPILOGUE_SWIGLU stores -- thresholding them with `tau` and listing the survivors as celty_spmspv does
 * (celty_last_compaction then reports that list, ascending).  No launch and no pass over memory sits between the
 * two products.  h_out_dev (may be NULL) receives the K FP16 values of x.  `ep` as in celty_spmspv_ex.
 * Errors: as celty_spmspv_ex.
 */
int celty_spmspv_swiglu(celty_matrix *m, const float *gate_up_dev, float tau, void *y_dev, void *h_out_dev,
                        const celty_epilogue *ep, celty_stream_t stream);

/*
 * celty_spmspv_host -- the same call for HOST vectors: copies x_host (K FP16) to x_stage_dev,
 * runs celty_spmspv into y_stage_dev, copies it to y_host (M FP32) and synchronises `stream`
 * before returning.  Use page-locked host memory for the copies to be asynchronous.
 * x_stage_dev (2K bytes) and y_stage_dev (4M bytes) are caller-provided device buffers.
 */
int celty_spmspv_host(celty_matrix *m, const void *x_host, float tau, void *y_host, void *x_stage_dev,
                      void *y_stage_dev, celty_stream_t stream);

/*
 * celty_spmspv_static -- the same product for callers that cannot allocate device memory.
 * (The paper has no counterpart: this entry point exists for deployment reasons only.)
 *
 * Some callers of this library run where cudaMalloc is not available to them: inside a stream
 * capture, under a memory pool that owns every byte of the device, in a plugin whose host forbids
 * allocations on its inference path.  celty_spmspv needs a caller-provided workspace for its
 * scratch (the compacted activation list); this variant keeps that scratch in a fixed array that
 * is part of the library image instead, so the caller passes only inputs and outputs:
 *   m          a LANE_TILE handle (host side only is used: sizes and table offsets)
 *   image_dev  the packed image on the device (image_bytes of celty_device_bytes; the caller
 *              copied celty_host_image there, or it is the buffer given to celty_bind_device)
 *   x_dev      K FP16 (device, 16-byte aligned), not modified
 *   y_dev      M FP32 (device, 16-byte aligned), overwritten
 * It runs the two-launch path (thresholding/compaction kernel, then the lane-tile SpMSpV kernel
 * that loads straight from global memory and merges with atomic adds) and calls no cudaMalloc,
 * cudaFree or other allocating routine.
 * Limit: K <= 32768 (the scratch array holds 196 864 bytes: a header, int32 indices and FP16 values
 * for that many columns; every GPU that loads the library carries it until the process exits);
 * larger K returns CELTY_ELIMIT.
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress, with that
 * device current); make that first call before any stream capture.
 * All calls on a device share the one array, which keeps the previous call's contents; nothing in it
 * has to start at zero (count and list are rewritten by every call), but two calls that overlap on
 * the GPU (different streams, or one stream of another thread) race on it: serialise them.
 * Errors: CELTY_EINVAL (null, misaligned, tau < 0 or not finite, COLUMN-layout handle), CELTY_ELIMIT,
 * CELTY_ECUDA.
 */
int celty_spmspv_static(const celty_matrix *m, const void *image_dev, const void *x_dev, float tau, void *y_dev,
                        celty_stream_t stream);

/*
 * celty_last_compaction -- device pointers into the handle's workspace holding the list the last
 * celty_spmspv produced (valid after that call's work on its stream has finished): |S|, indices,
 * FP16 values.  For parity tests and for byte accounting.
 */
int celty_last_compaction(const celty_matrix *m, const int32_t **count_dev, const int32_t **idx_dev,
                          const uint16_t **val_dev);

/*
 * celty_decode_device -- run the kernels' own run-length decoder (the device function the SpMSpV
 * kernel uses) on column `col` of the bound image and write, for each stored entry, in
 * the order of celty_decode_host, its absolute row and FP16 bit pattern (slots that exist only to
 * fill a 16-byte group are skipped).  rows_dev / vals_dev have room for cap entries;
 * count_dev[0] receives the number written.  For bit-exact decode parity tests.
 */
int celty_decode_device(celty_matrix *m, int64_t col, int32_t *rows_dev, uint16_t *vals_dev, int64_t cap,
                        int32_t *count_dev, celty_stream_t stream);

/*
 * celty_fetched_bytes -- algorithmic HBM bytes of one celty_spmspv call for a given surviving
 * column list (host array of n ascending indices): entry stream of those columns as laid out
 * (including alignment padding and per-block headers), their metadata words, x read once, the
 * list written, y written once.  Scratch traffic of the split-K merge is not counted.  Host-only
 * arithmetic on the handle's tables.
 */
int celty_fetched_bytes(const celty_matrix *m, const int32_t *idx_host, int64_t n, int64_t *stream_bytes,
                        int64_t *total_bytes);

/*
 * celty_stored_entries -- stored entries (kept weights + padding entries, Section 3.2) of the n listed
 * columns (host array of indices): times 2.5 bytes this is what the format itself makes a call fetch for
 * those columns, before any alignment padding or per-block header of the device image.  Host-only.
 * Errors: CELTY_EINVAL.
 */
int celty_stored_entries(const celty_matrix *m, const int32_t *idx_host, int64_t n, int64_t *entries);

/*
 * celty_layout_stats -- how evenly the LANE_TILE image loads the 32 lanes of a warp: the number of sub-blocks
 * (column, slab), the steps they take in total (a sub-block takes as many steps as its fullest lane has groups of 8
 * entries) and the groups they hold in total.  32 * steps / groups is how many step slots the kernel runs per
 * group that exists: 1 would be perfectly even lanes.  Host-only.  Errors: CELTY_EINVAL (COLUMN handle).
 */
int celty_layout_stats(const celty_matrix *m, int64_t *sub_blocks, int64_t *steps, int64_t *groups);

/*
 * celty_count_entries -- how many entries the format of Section 3.2 would store for a mask if its
 * runs were `run_bits` wide (1..8), whole columns, without building anything: the kept positions
 * (nnz) and the padding entries the rule inserts (a gap of g dropped rows costs floor(g / 2^run_bits)
 * of them; rows after a column's last kept row cost nothing).  An entry then takes 2 + run_bits / 8
 * bytes.  This is the quantity behind the paper's choice of 4-bit runs (Section 3.2, Figure 3); the
 * encoder itself takes 4 bits only.  mask_host: M x K row-major, `ldm` bytes from row to row,
 * nonzero = kept.  Host-only.  Errors: CELTY_EINVAL (null mask, M or K <= 0, ldm < K, run_bits
 * outside 1..8), CELTY_ENOMEM.
 */
int celty_count_entries(const uint8_t *mask_host, int64_t ldm, int64_t M, int64_t K, int run_bits, int64_t *nnz,
                        int64_t *n_pad);

/*
 * celty_last_status -- synchronises `stream`, reads the workspace status word and clears it.
 * Returns CELTY_OK, CELTY_ETIMEOUT or CELTY_EBOUNDS (or CELTY_ECUDA / CELTY_ESTATE).
 */
int celty_last_status(celty_matrix *m, celty_stream_t stream);

/*
 * celty_set_launch -- tuning knobs for experiments and tests; 0 = the library's choice.
 *   grid     thread blocks per launch (at most what fits the device at once, at least one per row part)
 *   variant  LANE_TILE only, a sum of: 1 = two launches (compaction kernel, then a kernel that loads
 *            straight from global memory) instead of the single fused launch; for the fused launch
 *            2 = merge the blocks' results through per-block partial vectors summed in a fixed
 *            order (bit-reproducible) instead of adding them into y with bulk reduce-add copies,
 *            4 = force the bulk reduce-add merge, 8 = plain launch instead of a programmatic dependent
 *            launch (with which the kernel's set-up overlaps the tail of the previous kernel of the stream),
 *            16 = always / 32 = never run warp pairs: two warps per team that take turns at the team's
 *            accumulator, one waiting for its next sub-block and reading its header while the other runs its
 *            steps (by default the library pairs warps where a team has a dozen or more columns to stream),
 *            64 = never / 128 = wherever possible share a thread block between row parts.  (With the bulk
 *            reduce-add merge and no clusters: when the blocks do not divide by the row parts and the blocks left
 *            over can be shared evenly, each of them can serve several parts with correspondingly fewer teams per
 *            part, instead of giving some parts one block more than others, which leaves those blocks idle at the
 *            end.  By default the library does so where the parts have few enough blocks each for that to pay.)
 *            256 = run the build of the fused kernel that has every option compiled in even where the launch is
 *            the default one (bulk reduce-add merge, no clusters), for which the library otherwise uses smaller
 *            builds without the other options' code (same results; the smaller builds are faster).
 *   groups   fused kernel: warp teams per slab working on different columns (each has an accumulator)
 *   depth    fused kernel: bulk copies each team keeps in flight (ring slots)
 *   cluster  fused kernel, bulk reduce-add merge: thread blocks per cluster (1, 2 or 4); the blocks of a
 *            cluster add their accumulators through distributed shared memory before anything goes to y
 *            (the split-K trade-off of Sections 3.1 and 6.4 with an on-chip stage).  A size the grid or the
 *            device cannot take is halved until it fits.
 * Errors: CELTY_EINVAL.
 */
int celty_set_launch(celty_matrix *m, int32_t grid, int32_t variant, int32_t groups, int32_t depth, int32_t cluster);

/*
 * celty_set_register_rows -- the register / shared-memory accumulation split (LANE_TILE, single-launch kernel).
 * The paper moves accumulation into the register file with new hardware (Section 4.1) and studies how much of it
 * to move (Section 6.4, "Register vs. SMEM accumulation tradeoff"); this is the software analogue on a stock SM.
 * The first `rows` local rows of every lane's tile (0, 32, 64, 96 or 128; 0 = all sums in shared memory, the
 * library's default) are summed in registers across all the columns a warp team works on: for such a row the
 * kernel stores the product value * x_j into the row's shared-memory cell without loading the cell first, and
 * after every column each lane adds its cells to statically indexed registers and clears them; the registers go
 * to shared memory once, before the merge.  Those builds run 256 threads per block (at most eight teams).
 * Measured slower than the default at every split (the per-column collection costs more shared-memory traffic
 * than the loads it saves); kept as the measured answer to that question.
 * Errors: CELTY_EINVAL.
 */
int celty_set_register_rows(celty_matrix *m, int32_t rows);

/*
 * celty_launch_plan -- the shape the fused kernel would be launched with for this handle on the current
 * device, with the knobs of celty_set_launch applied (LANE_TILE handles; needs a CUDA device):
 *   out[0..9] = thread blocks, threads per block, dynamic shared memory (bytes), warp teams per slab,
 *   ring slots per team, thread blocks per cluster, row parts, slabs per block, ring slot size (bytes),
 *   merge (0 ordered two-stage sum, 1 bulk reduce-add) + 16 if warp pairs are in use + 256 x the number of row
 *   parts a left-over block serves (1 = blocks are not shared between parts).   n = capacity of out (at least 10).
 * Errors: CELTY_EINVAL, CELTY_ECUDA.
 */
int celty_launch_plan(const celty_matrix *m, int32_t *out, int32_t n);

/*
 * celty_set_wait_limit -- how many polls a bounded wait inside the kernels (for a bulk copy, for the other
 * thread blocks' tickets) makes before it gives up, sets the status word and lets the kernel finish; 0 = the
 * library's limit (about two million polls, far beyond any real wait).  The kernels never spin without a
 * limit: a wait that runs out shows up as CELTY_ETIMEOUT from celty_last_status, the call's y is then
 * undefined, and the handle is usable again after that call to celty_last_status.
 * Errors: CELTY_EINVAL.
 */
int celty_set_wait_limit(celty_matrix *m, uint32_t polls);

/* The cudaError_t of the last failing CUDA call made through this library (0 if none). */
int celty_last_cuda_error(void);

/* Static string for a celty_status. */
const char *celty_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* CELTY_H */
