/*
 * libpatconv, third operation: a depthwise pattern-pruned 3x3 convolution layer on
 * NVIDIA B200 (sm_100a).
 *
 * The layer (paper Sec. 2.1, "Pattern-Based Pruning", which says the scheme generalises
 * beyond the dense 3x3 layer): every channel has ONE 3x3 kernel of its own; the kernel
 * keeps the 4 weights of one pattern of the library, or is removed altogether.  For
 * every n, oy, ox, c
 *
 *   y = act( bias[c] + sum_{t in pattern(c)} W[c][t] * x[n][oy*s + dy(t) - 1][ox*s + dx(t) - 1][c] )
 *
 * with t = 3*dy + dx, zero padding of 1, stride s in {1,2}, act = ReLU or identity.
 * Same conventions as patconv.h.
 */
#ifndef XGEN_DWCONV_H
#define XGEN_DWCONV_H

#include "patconv.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct xgen_dwconv_packed xgen_dwconv_packed; /* opaque; owns host and device memory */

typedef struct {
    int32_t channels;               /* >= 1                                                    */
    int32_t stride;                 /* 1 or 2                                                  */
    int32_t pad;                    /* must be 1                                               */
    xgen_dtype dtype;               /* XGEN_F32, or XGEN_F16_F32ACC (x, W, y fp16; bias and sums fp32) */
    int32_t num_patterns;           /* P, 1..126                                               */
    const uint16_t *pattern_masks;  /* [P] host; bit (3*dy+dx) set = tap kept; popcount 4      */
} xgen_dwconv_desc;

/*
 * Pack one layer (offline; Sec. 2.3: patterns are known after training).  The device copy
 * holds, per tap, one fp32 weight per channel with pruned taps stored as zeros: the layer is
 * bound by memory traffic on this GPU (4 useful multiply-adds per 2 activations moved), every
 * input element is needed by some channel's neighbour anyway, so nothing is gained by
 * skipping taps, and the kernel runs all nine with the masked weights.
 *   dense_w_host    [channels][3][3] fp32 or IEEE fp16 bits; values at pruned taps are ignored
 *   pattern_id_host [channels]: index into desc->pattern_masks, or -1 for a removed kernel
 *   device          CUDA device ordinal, or -1 for a host-only handle (cannot run)
 * Errors: INVALID_ARG, BAD_PATTERN, UNSUPPORTED (pad != 1, stride not 1|2, dtype), ALLOC, CUDA.
 */
xgen_status xgen_dwconv_pack(const xgen_dwconv_desc *desc, const void *dense_w_host,
                             const int16_t *pattern_id_host, int device, xgen_dwconv_packed **out);

/*
 * Run the layer (Sec. 2.2: bias and ReLU fused).
 *   x_dev    [n][h][w][channels] NHWC, element-aligned
 *   bias_dev [channels] fp32 or NULL
 *   y_dev    [n][ho][wo][channels] NHWC, ho = (h + 2 - 3)/stride + 1, likewise wo; must not
 *            overlap x_dev
 * With channels a multiple of 4 and x_dev, y_dev 16-byte aligned (8-byte for fp16) a thread
 * moves four channels per access; otherwise one.  Only enqueues one kernel on the stream.
 * Errors: INVALID_ARG, SHAPE (n,h,w < 1 or a tensor beyond 2^31-1 elements), CUDA.
 */
xgen_status xgen_dwconv_run(const xgen_dwconv_packed *packed, const void *x_dev, int32_t n, int32_t h,
                            int32_t w, const void *bias_dev, int32_t relu, void *y_dev, void *cuda_stream);

/* Number of channels whose kernel survives (4 useful multiply-adds per output element each). */
xgen_status xgen_dwconv_query(const xgen_dwconv_packed *packed, int64_t *kernels_surviving);

/* Release the handle and its device memory.  NULL is allowed. */
void xgen_dwconv_free(xgen_dwconv_packed *packed);

#ifdef __cplusplus
}
#endif
#endif /* XGEN_DWCONV_H */
