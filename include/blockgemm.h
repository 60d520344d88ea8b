/*
 * libpatconv, second operation: inference-time execution of a block-pruned
 * matrix product on NVIDIA B200 (sm_100a) -- a fully connected layer, or a 1x1
 * convolution taken in its matrix form.
 *
 * The layer (paper Sec. 2.1, "Block-Based Pruning"): the weight matrix W
 * [c_out][k] is cut into equal blocks of block_rows x block_cols entries, and in
 * every block whole rows and whole columns are pruned, independently of the
 * other blocks.  An entry survives if its row and its column are both kept in
 * its block.  For every row m of the input and every output channel oc
 *
 *   y[m][oc] = act( bias[oc] + sum_{c: W[oc][c] survives} W[oc][c] * x[m][c] )
 *
 * with x [m_rows][k] row-major (one row per pixel of an NHWC activation tensor,
 * m_rows = n*h*w, or one row per token) and act = ReLU or identity.
 *
 * Same conventions as patconv.h: plain C ABI, every function returns a status,
 * *_host is host memory, *_dev memory of the device the handle was packed for.
 */
#ifndef XGEN_BLOCKGEMM_H
#define XGEN_BLOCKGEMM_H

#include "patconv.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct xgen_blockgemm_packed xgen_blockgemm_packed; /* opaque; owns host and device memory */

typedef struct {
    int32_t k;              /* input features (columns of W), >= 1                         */
    int32_t c_out;          /* output channels (rows of W), >= 1                           */
    int32_t block_rows;     /* rows of a pruning block, >= 1 (blocks at the bottom edge may be smaller) */
    int32_t block_cols;     /* columns of a pruning block, >= 1 (likewise at the right edge) */
    xgen_dtype dtype;       /* XGEN_F32 (x, W, y fp32) or XGEN_F16_F32ACC (x, W, y IEEE fp16, bias
                               fp32, sums in fp32, one round-to-nearest-even at the store)  */
    int32_t warps_per_block; /* tuning-decided (paper Sec. 2.3: the layerwise representation carries
                               such parameters): warps of a thread block, 16 output channels each;
                               0 = the library's choice, else 1..16.  Fewer warps make smaller
                               thread blocks, of which an SM holds several at a time            */
} xgen_blockgemm_desc;

/* What xgen_blockgemm_query reports. */
typedef struct {
    int64_t weights_total;      /* k * c_out                                                     */
    int64_t weights_kept;       /* entries whose row and column are kept in their block = useful
                                   multiply-adds per row of x                                     */
    int64_t weight_bytes;       /* bytes of the kept weights at the layer's storage precision    */
    int64_t stream_bytes;       /* bytes of the packed stream on the device (every kept weight
                                   widened to fp32; headers, padding and the offset table included) */
    int64_t padded_slots;       /* weight slots of the stream that hold padding zeros (a column
                                   group is filled up to eight columns)                          */
    int64_t column_groups;      /* activation loads in the stream: one per group of up to eight
                                   kept columns of a block, per warp that has kept rows there    */
    int64_t row_commands;       /* (kept row, column group) pairs: one command each              */
    int32_t rows_per_warp;      /* output channels one warp accumulates (16)                     */
    int32_t warps_per_block;
    int32_t row_blocks;         /* thread blocks along c_out                                     */
    int32_t stage_cols;         /* input columns staged per pipeline step                        */
    int32_t n_stages;
    int32_t max_stage_bytes;    /* largest per-(thread block, stage) piece of the stream         */
} xgen_blockgemm_stats;

/*
 * Pack one layer (paper Sec. 2.1, "Block-Based Pruning": the block structure and what is
 * pruned in each block are known after training, so the kept entries are compacted offline).
 *   dense_w_host   [c_out][k] fp32 (XGEN_F32) or IEEE fp16 bits (XGEN_F16_F32ACC).  Values at
 *                  pruned positions are ignored; they need not be zero.
 *   row_keep_host  [ceil(c_out/block_rows)][ceil(k/block_cols)][block_rows] bytes: non-zero =
 *                  this row of the block is kept (entries for rows beyond c_out are ignored)
 *   col_keep_host  [ceil(c_out/block_rows)][ceil(k/block_cols)][block_cols] bytes, likewise
 *   device         CUDA device ordinal to upload to, or -1 to build the host layout only (no
 *                  CUDA call is made; such a handle cannot run)
 *   out            receives the handle; release it with xgen_blockgemm_free
 * Synchronous.  Inputs are copied.  Errors: INVALID_ARG, UNSUPPORTED (dtype), SHAPE, ALLOC, CUDA.
 */
xgen_status xgen_blockgemm_pack(const xgen_blockgemm_desc *desc, const void *dense_w_host,
                                const uint8_t *row_keep_host, const uint8_t *col_keep_host,
                                int device, xgen_blockgemm_packed **out);

/*
 * Run the layer (paper Sec. 2.1: only the kept rows and columns of every block are computed;
 * Sec. 2.2: bias and ReLU fused).
 *   x_dev    [m_rows][k] row-major, the dtype's activation type, element-aligned (fp16: an
 *            even k and 4-byte alignment let the rows be staged by asynchronous copies;
 *            otherwise they are staged with plain loads)
 *   bias_dev [c_out] fp32, 4-byte aligned, or NULL
 *   y_dev    [m_rows][c_out] row-major, element-aligned, must not overlap x_dev (16-byte
 *            alignment and a row of a multiple of 16 bytes give 16-byte stores)
 *   cuda_stream  a cudaStream_t passed as void* (NULL = default stream)
 * Only enqueues one kernel on the stream: no synchronisation, no device allocation.
 * Errors: INVALID_ARG (null or misaligned pointer, overlap), SHAPE (m_rows < 1 or a tensor
 * beyond 2^31-1 elements), CUDA (launch failure or host-only handle).
 */
xgen_status xgen_blockgemm_run(const xgen_blockgemm_packed *packed, const void *x_dev, int64_t m_rows,
                               const void *bias_dev, int32_t relu, void *y_dev, void *cuda_stream);

/* Fill *stats (see xgen_blockgemm_stats). */
xgen_status xgen_blockgemm_query(const xgen_blockgemm_packed *packed, xgen_blockgemm_stats *stats);

/*
 * Read-only view of the packed stream on the host, for inspection and tests.  All pointers
 * belong to the handle.  The stream is an array of 16-byte units (4 words).  The commands of
 * warp w of the thread block for output channels [rb*16*warps_per_block, ...) in stage s
 * (input columns [s*stage_cols, ...)) are the units seg_off[(rb*n_stages + s)*(warps_per_block
 * + 1) + w] up to the next entry; warp w owns the block's channels 16*w .. 16*w + 15.  They are
 * a sequence of column groups:
 *   1 unit   {number of row commands, columns 0..3, columns 4..7, 0}: eight column numbers, one
 *            byte each, relative to the stage's first column; stage_cols marks a padding slot
 *   then per kept row 3 units: {16-byte header whose first word is 8 x (channel - the warp's
 *            first channel)}, {weights of columns 0..3}, {weights of columns 4..7} as fp32 bits
 *            (fp16 weights widened exactly; 0 in padding slots)
 */
typedef struct {
    const uint32_t *units;   int64_t n_units;
    const int32_t  *seg_off; /* [row_blocks * n_stages * (warps_per_block + 1)] */
} xgen_blockgemm_host_view;

/* Fill *view with pointers into the handle's host copy of the packed stream. */
xgen_status xgen_blockgemm_view(const xgen_blockgemm_packed *packed, xgen_blockgemm_host_view *view);

/* Release the handle and its device memory.  NULL is allowed. */
void xgen_blockgemm_free(xgen_blockgemm_packed *packed);

#ifdef __cplusplus
}
#endif
#endif /* XGEN_BLOCKGEMM_H */
