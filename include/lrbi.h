/*
 * lrbi -- inference with a layer pruned by a tiled low-rank binary index (B200, sm_100a).
 *
 * Plain C ABI.  The pruning index of a layer W [rows x cols] (rows = output features,
 * cols = input features) is not stored; it is rebuilt from two small binary factors per
 * tile.  The index matrix is cut into equal tiles of tile_rows x tile_cols (Section 3.1
 * of the paper: each block is factorised, hence decoded, independently, all with the same
 * rank k).  For tile (tr, tc) with factors Ip (tile_rows x k) and Iz (k x tile_cols) the
 * decoded index is the Boolean matrix product of Eq. 3,
 *
 *        Ia[i][j] = OR_{l=1..k} ( Ip[i][l] AND Iz[l][j] ),
 *
 * where a 1 keeps the weight and a 0 prunes it to zero (Section 2, Eq. 1-2).  Ia is the
 * masking layer of the layer (Sections 2 and 2.2), so the layer computes
 * Y = X * (W .* Ia)^T.
 *
 * Packed factor format (KW = ceil(k / 32) 32-bit words per row of Ip / per column of Iz,
 * GR = ceil(rows / tile_rows), GC = ceil(cols / tile_cols), tile index t = tr * GC + tc):
 *
 *   ip[(t * tile_rows + i) * KW + w]   bit (l % 32) of word w = l / 32   is  Ip_t[i][l]
 *   iz[(t * tile_cols + j) * KW + w]   bit (l % 32) of word w = l / 32   is  Iz_t[l][j]
 *
 * Edge tiles still hold tile_rows row words and tile_cols column words; those that fall
 * outside the matrix are ignored.  Bits at positions >= k of the last word are ignored.
 *
 * Unless an argument says "host", every pointer is a DEVICE pointer owned by the caller,
 * valid on the current device, 16-byte aligned.  Calls are asynchronous and ordered on
 * `stream` (a cudaStream_t passed as void*, NULL = the legacy default stream).  Inputs are
 * only read.  Nothing outside the stated output extent is written.  Argument errors are
 * detected on the host before anything is launched and reported by the return code; no
 * call aborts, throws or traps.  There is no CPU fallback: without a usable sm_100 device
 * a compute call returns LRBI_ERR_CUDA.
 *
 * Timeouts.  Every wait inside a kernel is bounded (about two seconds); a wait that runs out
 * leaves a code in a per-device status word, the kernel ends early and its output is
 * incomplete.  The asynchronous calls (lrbi_decode_mask, lrbi_masked_gemm, ..._static) cannot
 * know this when they return.  The contract is: a call that synchronises
 * (lrbi_layer_forward_host, lrbi_device_status, lrbi_last_device_error) reads the word; once
 * it has been seen non-zero, every compute call on that device returns LRBI_ERR_TIMEOUT and
 * launches nothing until lrbi_device_status(1) clears it.  A caller of the asynchronous calls
 * checks lrbi_device_status after synchronising its stream.
 *
 * Threads.  Entry points may be called from several host threads; the library's own lazily
 * built state is guarded by one lock.  Two calls that use the K-split buffer of
 * lrbi_masked_gemm (or the fixed array of lrbi_masked_gemm_static) at the same time on
 * different streams race on the device: order them.
 *
 * Non-finite values.  A NaN/Inf stored in a PRUNED weight never reaches Y (the weight is
 * selected away).  Activations must be finite: the tensor-core kernels zero the pruned weight
 * and still multiply, so an Inf/NaN in X at a pruned column gives NaN there, while the
 * CUDA-core kernels skip the product; which kernel runs depends on the batch.
 */
#ifndef LRBI_H_
#define LRBI_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define LRBI_API __attribute__((visibility("default")))
#else
#define LRBI_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    LRBI_OK = 0,
    LRBI_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, misaligned pointer          */
    LRBI_ERR_UNSUPPORTED = 2, /* a shape, dtype or kernel choice this library does not cover   */
    LRBI_ERR_CUDA = 3,        /* a CUDA runtime/driver call failed (see lrbi_last_cuda_error)  */
    LRBI_ERR_TIMEOUT = 4,     /* a bounded device-side wait gave up earlier on this device and has
                                 been seen by a synchronising call; cleared by lrbi_device_status(1) */
    LRBI_ERR_TOO_LARGE = 5    /* the problem needs more fixed scratch than the library carries   */
} lrbi_status;

/* Geometry of one pruned layer (Section 3.1: equal tiles, one rank). */
typedef struct {
    int32_t rows;      /* output features: rows of W and of the index          */
    int32_t cols;      /* input features: columns of W and of the index        */
    int32_t tile_rows; /* tm >= 1                                               */
    int32_t tile_cols; /* tn >= 1                                               */
    int32_t rank;      /* k >= 1, the same for every tile                       */
} lrbi_layout;

/* Output element type of lrbi_masked_gemm. */
enum { LRBI_Y_BF16 = 0, LRBI_Y_F32 = 1 };

/* Kernel choice for lrbi_masked_gemm / lrbi_decode_mask (LRBI_ALGO_AUTO picks by shape). */
enum {
    LRBI_ALGO_AUTO = 0,
    LRBI_ALGO_GENERIC = 1,   /* any shape; one thread per output, slow                         */
    LRBI_ALGO_GEMV = 2,      /* small batch, bandwidth-bound, CUDA-core FMA                    */
    LRBI_ALGO_TENSOR = 3,    /* tcgen05 MMA with TMEM accumulators                             */
    LRBI_ALGO_DECODE_BALLOT = 4, /* decode: one __ballot_sync per 32-bit mask word             */
    LRBI_ALGO_DECODE_PLANES = 5, /* decode: Iz transposed into bit-planes, OR per 32 columns (variant by size) */
    LRBI_ALGO_DECODE_PLANES_WIDE = 6, /* decode: the 1024-column bit-plane variant, whatever the mask size */
    LRBI_ALGO_STREAM = 7,    /* batch <= 32, bandwidth-bound, warp-level tensor-core MMAs              */
    /* The next two force an instantiation that LRBI_ALGO_TENSOR otherwise picks from the problem size
       (any shape LRBI_ALGO_TENSOR covers; small problems just leave most of a tile empty). */
    LRBI_ALGO_TENSOR_PAIR = 8,  /* tcgen05 CTA pairs (cta_group::2), 256 rows x 256 batch rows per pair  */
    LRBI_ALGO_TENSOR_PAIR2 = 9, /* CTA pairs with two accumulators: 256 rows x 512 batch rows per pair   */
    LRBI_ALGO_TENSOR_PAIR192 = 10 /* CTA pairs, one accumulator of 192 batch rows (few rows, long batch)   */
};

/* Element counts of the packed arrays for a layout (0 if the layout is invalid). */
LRBI_API size_t lrbi_packed_ip_words(const lrbi_layout *layout); /* GR*GC*tile_rows*KW */
LRBI_API size_t lrbi_packed_iz_words(const lrbi_layout *layout); /* GR*GC*tile_cols*KW */
LRBI_API size_t lrbi_mask_words(const lrbi_layout *layout);      /* rows*ceil(cols/32) */

/*
 * Decode the whole index (Eq. 3 per tile, Section 3.1) into a bit-packed mask.
 *   ip, iz    device, packed factors as above (read only)
 *   mask_out  device, rows x ceil(cols/32) uint32, row-major; bit (c % 32) of word c / 32
 *             of row r is Ia[r][c]; bits beyond `cols` in the last word of a row are 0.
 *   algo      LRBI_ALGO_AUTO, LRBI_ALGO_DECODE_BALLOT, LRBI_ALGO_DECODE_PLANES (needs
 *             tile_cols % 32 == 0) or LRBI_ALGO_DECODE_PLANES_WIDE (needs rank <= 256 and tiles of 128, 256,
 *             512 or a multiple of 1024 columns, or a single tile column of a multiple of 128 columns);
 *             a variant that does not cover the layout returns LRBI_ERR_UNSUPPORTED
 * Every word of mask_out is written; nothing else is.
 */
LRBI_API lrbi_status lrbi_decode_mask(const lrbi_layout *layout, const uint32_t *ip, const uint32_t *iz,
                             uint32_t *mask_out, int32_t algo, void *stream);

/*
 * Fused decode + prune + dense product (Eq. 3; masking layer of Sections 2 and 2.2):
 *       Y[b][o] = sum_i  Ia[o][i] ? X[b][i] * W[o][i] : 0      (fp32 accumulation)
 * The decoded index never reaches device memory.  A pruned weight is selected away (its bf16
 * pattern is replaced by +0 or its product is skipped), so a NaN/Inf stored in a pruned
 * position does not reach Y.  X must be finite (see "Non-finite values" above).
 *   W      device, bf16 bit patterns, [rows][cols] row-major
 *   X      device, bf16 bit patterns, [batch][cols] row-major
 *   Y      device, [batch][rows] row-major, bf16 (round to nearest even) or fp32 per y_dtype
 *   algo   LRBI_ALGO_AUTO, _GENERIC, _GEMV (batch <= 8), _STREAM (batch <= 32), _TENSOR, _TENSOR_PAIR or
 *          _TENSOR_PAIR2 / _TENSOR_PAIR192; a kernel that does not
 *          cover the shape returns LRBI_ERR_UNSUPPORTED and launches nothing.
 * The tensor-core path may split the reduction over several thread blocks; it then keeps
 * fp32 partial sums in a library-owned device buffer that grows (cudaMalloc) on the first
 * call that needs more, so such a first call must not be made during stream capture.
 * Calls that use that buffer concurrently on different streams are not supported.
 */
LRBI_API lrbi_status lrbi_masked_gemm(const lrbi_layout *layout, const uint16_t *W, const uint32_t *ip,
                             const uint32_t *iz, const uint16_t *X, int32_t batch, void *Y,
                             int32_t y_dtype, int32_t algo, void *stream);

/*
 * lrbi_masked_gemm for callers that must not allocate device memory.  (The paper has no
 * counterpart to this call; it exists for the library's users.)
 *
 * Who needs it: code that runs inside a memory-pool or arena discipline where every device byte
 * is accounted for up front (an inference server that sizes its pool at start-up and treats a
 * later cudaMalloc as a bug), code that runs where cudaMalloc may block or fail at a bad moment
 * (it takes a device-wide lock and can synchronise; under memory pressure it returns an error in
 * the middle of a request), and plug-ins that are simply not given the right to allocate.
 * lrbi_masked_gemm may allocate: when it splits the reduction over K it keeps fp32 partial sums
 * in a buffer that it grows with cudaMalloc.  This call never does.  It always runs the
 * tensor-core kernel (LRBI_ALGO_TENSOR shapes only, else LRBI_ERR_UNSUPPORTED) and keeps the
 * partial sums in a fixed array that is part of the library image: LRBI_STATIC_SCRATCH_BYTES
 * (8 MiB) of device memory on every GPU that loads the library, held until the process exits.
 *
 *   - If splits * batch * rows * 4 bytes exceeds that array the call returns LRBI_ERR_TOO_LARGE
 *     and launches nothing (lrbi_masked_gemm_static_bytes tells the need in advance; 0 = no
 *     scratch needed).  Problems with enough output tiles to fill the GPU do not split K and need none.
 *   - It calls no cudaMalloc, cudaFree or any other allocating routine.
 *   - The first call on a device looks up the array's device address (once per device, with that
 *     device current) and caches it; make that first call before starting any stream capture.
 *   - All calls on a device share the one array, and it keeps whatever the last call left in it.
 *     Nothing has to be cleared: every word the reduction reads was written earlier in the same
 *     call.  But two calls that overlap on the GPU (different streams) race on it and give wrong
 *     results: keep calls to this entry point on one stream, or order them with events.
 * Arguments, layouts and results are those of lrbi_masked_gemm with LRBI_ALGO_TENSOR.
 */
#define LRBI_STATIC_SCRATCH_BYTES (8u * 1024u * 1024u)
LRBI_API lrbi_status lrbi_masked_gemm_static(const lrbi_layout *layout, const uint16_t *W, const uint32_t *ip,
                                             const uint32_t *iz, const uint16_t *X, int32_t batch, void *Y,
                                             int32_t y_dtype, void *stream);
LRBI_API size_t lrbi_masked_gemm_static_bytes(const lrbi_layout *layout, int32_t batch);

/*
 * Same computation for callers whose activations live in host memory (the index and the
 * weights are uploaded once, activations and results cross the bus on every call).
 *   lrbi_layer_create   copies W, ip, iz (HOST pointers) to the current device and reserves
 *                       staging for up to max_batch rows.  *out owns device memory.
 *   lrbi_layer_forward_host   X_host [batch][cols] bf16 and Y_host [batch][rows] are HOST
 *                       pointers (pinned memory makes the copies asynchronous and overlapped
 *                       with the kernels, chunk by chunk); returns after Y_host is complete.
 *   lrbi_layer_destroy  frees everything the handle owns.
 */
typedef struct lrbi_layer lrbi_layer;
LRBI_API lrbi_status lrbi_layer_create(const lrbi_layout *layout, const uint16_t *W_host,
                              const uint32_t *ip_host, const uint32_t *iz_host,
                              int32_t max_batch, lrbi_layer **out);
LRBI_API lrbi_status lrbi_layer_forward_host(lrbi_layer *layer, const uint16_t *X_host, int32_t batch,
                                    void *Y_host, int32_t y_dtype, int32_t algo);
LRBI_API lrbi_status lrbi_layer_destroy(lrbi_layer *layer);

/*
 * Inner loop of Algorithm 1 (Section 2.1: "binary pruning-index-data matrix factorization").  The NMF of
 * |W| and the search over S_p stay with the caller; these two calls are the steps the search repeats.
 *
 * lrbi_threshold_pack: binary conversion of the NMF factors (the sentence under Eq. 4; Eq. 4 -> Eq. 5),
 *       (Ip)[i][l] = 1 if (Mp)[i][l] >= T_p else 0,     (Iz)[l][j] = 1 if (Mz)[l][j] >= T_z else 0,
 * written in the packed factor format above.  Every tile is its own factorisation (Section 3.1) and has its
 * own pair of thresholds.
 *   mp   device, fp32, [GR*GC][tile_rows][rank]   row-major per tile
 *   mz   device, fp32, [GR*GC][rank][tile_cols]   row-major per tile
 *   tp, tz   device, fp32, [GR*GC]   thresholds of each tile (+inf gives an empty factor)
 *   ip_out, iz_out   device, lrbi_packed_ip_words / lrbi_packed_iz_words words; bits >= rank are written as 0
 *
 * lrbi_index_cost: what the search looks at for one candidate (ip, iz), per tile, tiles in row-major grid order:
 *   kept_i = number of ones of the magnitude index I = (|W| >= theta)            (Eq. 1 -> Eq. 2)
 *   kept_a = number of ones of the decoded index Ia = Ip (x) Iz                  (Eq. 3; S_a = 1 - kept_a / size)
 *   lost   = number of positions with I = 1 and Ia = 0
 *   cost   = sum of |W| over those positions                                    (the Cost line of Algorithm 1)
 * W is read once, Ia is decoded on the fly and never stored.  A NaN weight counts as pruned (I = 0).  cost is
 * summed in fp32 per 8 weights and in fp64 beyond; blocks add to a tile's record with atomics, so the last bits
 * of cost may differ between calls.
 *   W    device, bf16 bit patterns, [rows][cols]
 *   out  device, GR*GC records, 8-byte aligned; overwritten
 * Only positions inside the matrix are counted (edge tiles are smaller).
 */
typedef struct {
    uint64_t kept_i;
    uint64_t kept_a;
    uint64_t lost;
    double cost;
} lrbi_tile_cost;
LRBI_API lrbi_status lrbi_threshold_pack(const lrbi_layout *layout, const float *mp, const float *mz, const float *tp,
                                         const float *tz, uint32_t *ip_out, uint32_t *iz_out, void *stream);
LRBI_API lrbi_status lrbi_index_cost(const lrbi_layout *layout, const uint16_t *W, float theta, const uint32_t *ip,
                                     const uint32_t *iz, lrbi_tile_cost *out, void *stream);

/*
 * Generalised layouts (Section 3.1, last paragraph: "each submatrix can optimally choose a different rank").
 *
 * Ranked layout: tile t (row-major grid order) has its own rank k_t, 0 <= k_t <= layout->rank (the layout's rank is
 * then only the upper bound), and is packed with KW_t = ceil(k_t / 32) words per row of Ip / column of Iz:
 *       ip[ip_offset[t] + i * KW_t + w],      iz[iz_offset[t] + j * KW_t + w]
 * so a tile of low rank takes less room (k_t (tile_rows + tile_cols) bits, the index size of Section 2 for that
 * tile).  A tile of rank 0 is empty: everything in it is pruned.  The three arrays are DEVICE arrays of GR*GC
 * entries; offsets count 32-bit words.  Tile bases need only 4-byte alignment.
 *   lrbi_decode_mask_ranked   Eq. 3 per tile with the tile's rank -> bit-packed mask (as lrbi_decode_mask)
 *   lrbi_masked_gemm_ranked   the fused product (as lrbi_masked_gemm); the tensor-core kernel runs when the shape
 *                             allows it (LRBI_ALGO_TENSOR's conditions), else a one-thread-per-output kernel
 *
 * lrbi_decode_mask_batch: the indices of n layers decoded by ONE launch per 32 layers (many small layers, e.g. the
 * blocks of a network, cost one launch latency instead of n).  layouts, ip, iz, mask_out are HOST arrays of n
 * entries; the pointers they hold are device pointers as for lrbi_decode_mask.
 */
typedef struct {
    const int32_t *ranks;     /* device, [GR*GC]                                   */
    const int64_t *ip_offset; /* device, [GR*GC], first word of tile t in ip       */
    const int64_t *iz_offset; /* device, [GR*GC], first word of tile t in iz       */
} lrbi_tile_ranks;
LRBI_API lrbi_status lrbi_decode_mask_ranked(const lrbi_layout *layout, const lrbi_tile_ranks *ranks, const uint32_t *ip,
                                             const uint32_t *iz, uint32_t *mask_out, void *stream);
LRBI_API lrbi_status lrbi_masked_gemm_ranked(const lrbi_layout *layout, const lrbi_tile_ranks *ranks, const uint16_t *W,
                                             const uint32_t *ip, const uint32_t *iz, const uint16_t *X, int32_t batch,
                                             void *Y, int32_t y_dtype, int32_t algo, void *stream);
LRBI_API lrbi_status lrbi_decode_mask_batch(int32_t n, const lrbi_layout *layouts, const uint32_t *const *ip,
                                            const uint32_t *const *iz, uint32_t *const *mask_out, void *stream);

/*
 * NMF of the magnitude matrix (Section 2.1: M[i][j] = |W[i][j]| "is factorized by an NMF library" into Mp, Mz,
 * Eq. 4; first two steps of Algorithm 1), every tile on its own (Section 3.1).  The paper names no solver; this is
 * the multiplicative update rule for the Frobenius objective ||M - Mp Mz||^2 of the NMF reference it cites, from
 * the caller's starting factors: per iteration
 *       Mz <- Mz * (Mp^T M) / (Mp^T Mp Mz + eps),   then   Mp <- Mp * (M Mz^T) / (Mp Mz Mz^T + eps),
 * in fp32.  Positions of an edge tile outside the matrix count as zeros of M.  rank <= 256.
 *   W     device, bf16 bit patterns, [rows][cols]
 *   mp    device, fp32, [GR*GC][tile_rows][rank], in and out (start from positive values)
 *   mz    device, fp32, [GR*GC][rank][tile_cols], in and out
 *   workspace   device, lrbi_nmf_workspace(layout) bytes, 16-byte aligned, scratch for the call
 * The results feed lrbi_threshold_pack.
 */
LRBI_API size_t lrbi_nmf_workspace(const lrbi_layout *layout);
LRBI_API lrbi_status lrbi_nmf_update(const lrbi_layout *layout, const uint16_t *W, float *mp, float *mz, int32_t iterations,
                                     float eps, void *workspace, size_t workspace_bytes, void *stream);

/*
 * Backward pass of the masked layer (Section 2.2: the pruned network is retrained "using a masking layer" Ia, so
 * gradients flow through kept weights only).  With Y = X (W .* Ia)^T and dY = dL/dY [batch][rows]:
 *       dX[b][i] = sum_o  Ia[o][i] ? dY[b][o] * W[o][i] : 0          dW[o][i] = Ia[o][i] ? sum_b dY[b][o] * X[b][i] : 0
 * fp32 accumulation; outputs bf16 (round to nearest even) or fp32 as the dtype argument says (LRBI_Y_*).
 *
 * lrbi_masked_gemm_dx   needs the weights TRANSPOSED: Wt [cols][rows] bf16 (keep that copy beside W and refresh it with
 *       lrbi_transpose_bf16 when W changes).  It is the forward product of the transposed layer, so it runs on the same
 *       kernels: the packed factors are used as they are (a row word of Ip is a column word of Ip^T).  algo:
 *       LRBI_ALGO_AUTO, _GENERIC or _TENSOR / _TENSOR_PAIR / _TENSOR_PAIR2 / _TENSOR_PAIR192 (tensor-core shapes: rows % 8 == 0, and
 *       tile_cols % 128 == 0 and tile_rows % 64 == 0 unless the grid has one tile in that direction).
 * lrbi_masked_gemm_dw   dY [batch][rows], X [batch][cols] -> dW [rows][cols].  Large aligned layers (rows, cols and
 *       batch multiples of 8; tile_cols % 128 == 0 and tile_rows % 256 == 0 unless the grid has one tile in that
 *       direction) run as ONE launch of the tensor-core kernel on dY and X as they are (the operands are read
 *       MN-major): nothing is pruned inside the contraction and the index, decoded on the fly and never stored, is
 *       applied as dW is written; `workspace` is not touched and may be NULL.  Other tensor-core shapes use
 *       `workspace` (DEVICE memory of at least lrbi_masked_gemm_dw_workspace(layout, batch) bytes, 16-byte aligned,
 *       owned by the caller, scratch for the call) for transposed copies of dY and X and apply the index to dW in
 *       place afterwards; batch % 8 != 0, or a NULL workspace on such a shape, falls back to a slow
 *       one-thread-per-weight kernel.
 * lrbi_transpose_bf16   dst [cols][rows] = transpose of src [rows][cols] (bf16 bit patterns; dst must not overlap src).
 */
LRBI_API lrbi_status lrbi_transpose_bf16(const uint16_t *src, int32_t rows, int32_t cols, uint16_t *dst, void *stream);
LRBI_API lrbi_status lrbi_masked_gemm_dx(const lrbi_layout *layout, const uint16_t *Wt, const uint32_t *ip, const uint32_t *iz,
                                         const uint16_t *dY, int32_t batch, void *dX, int32_t dx_dtype, int32_t algo, void *stream);
LRBI_API size_t lrbi_masked_gemm_dw_workspace(const lrbi_layout *layout, int32_t batch);
LRBI_API lrbi_status lrbi_masked_gemm_dw(const lrbi_layout *layout, const uint16_t *dY, const uint16_t *X, int32_t batch,
                                         const uint32_t *ip, const uint32_t *iz, void *dW, int32_t dw_dtype,
                                         void *workspace, size_t workspace_bytes, void *stream);

/* Which kernel LRBI_ALGO_AUTO would run for this layout and batch (an LRBI_ALGO_* value). */
LRBI_API int32_t lrbi_masked_gemm_choice(const lrbi_layout *layout, int32_t batch);

/*
 * How lrbi_masked_gemm would run a call on the current device (nothing is launched).  For
 * LRBI_ALGO_TENSOR the fields say which instantiation of the tcgen05 kernel runs; for the other
 * kernels only `algo` is meaningful (k_splits = 1, the rest 0).
 */
typedef struct {
    int32_t algo;          /* the LRBI_ALGO_* value that runs (LRBI_ALGO_AUTO resolved)             */
    int32_t batch_tile;    /* batch rows per output tile (512: a CTA pair with two accumulators)    */
    int32_t cta_pair;      /* 1: two CTAs of a cluster share a 256-row tile (tcgen05 cta_group::2)  */
    int32_t panel_columns; /* columns of the index decoded per step inside the kernel (256 or 64)   */
    int32_t k_splits;      /* thread blocks along the reduction; > 1 means fp32 partial sums + a second kernel */
    int32_t stages;        /* operand stages in shared memory                                       */
    uint64_t scratch_bytes;/* bytes of partial sums (what lrbi_masked_gemm_static_bytes reports)    */
} lrbi_gemm_plan;
LRBI_API lrbi_status lrbi_masked_gemm_plan(const lrbi_layout *layout, int32_t batch, int32_t algo,
                                           lrbi_gemm_plan *plan);

/* Kernels launched by this library since it was loaded (all entry points, this process). */
LRBI_API uint64_t lrbi_launch_count(void);

/*
 * Device-side status word of the current device: 0, or a code left by a kernel whose bounded
 * wait (pipeline barrier) ran out.  Synchronises the device.  `clear` != 0 resets it and
 * lifts the LRBI_ERR_TIMEOUT refusal of later calls.  Returns -1 if a CUDA call failed.
 */
LRBI_API int32_t lrbi_device_status(int32_t clear);
LRBI_API int32_t lrbi_last_device_error(void); /* lrbi_device_status(0) */

/*
 * Self-test of the timeout path (no counterpart in the paper).  Launches one tiny kernel whose single
 * thread waits, with the same bounded wait the pipeline kernels use but a limit of `limit_us`
 * microseconds (at most 100 000), on a barrier that nothing signals.  The wait gives up, the kernel
 * returns normally and the status word of the device then holds 0x600.  Nothing hangs or traps; it is
 * how the tests show that a timeout is recorded, reported (LRBI_ERR_TIMEOUT) and cleared.
 */
LRBI_API lrbi_status lrbi_selftest_bounded_wait(uint32_t limit_us, void *stream);

LRBI_API const char *lrbi_status_string(lrbi_status s);
LRBI_API int32_t lrbi_last_cuda_error(void); /* cudaError_t / CUresult of the last failed call, else 0 */

#ifdef __cplusplus
}
#endif
#endif /* LRBI_H_ */
