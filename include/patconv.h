/*
 * libpatconv -- inference-time execution of a pattern-pruned 3x3 convolution
 * layer on NVIDIA B200 (sm_100a).
 *
 * The layer (paper Sec. 2.1, "Pattern-Based Pruning"): every surviving 3x3
 * kernel keeps the 4 weights of one shape out of a small library of pre-defined
 * patterns; connectivity pruning removes whole kernels, i.e. cuts the link
 * between one input and one output channel.  For every n, oy, ox, oc
 *
 *   y = act( bias[oc] + sum_{ic: kernel (oc,ic) survives} sum_{t in pattern(oc,ic)}
 *                          W[oc][ic][t] * x[n][oy*s + dy(t) - 1][ox*s + dx(t) - 1][ic] )
 *
 * with t = 3*dy + dx, zero padding of 1, stride s in {1,2}, cross-correlation
 * (no kernel flip), act = ReLU or identity.
 *
 * Plain C ABI: pointers and sizes only.  Every function returns a status code;
 * nothing throws, aborts or traps.  Unless stated otherwise a pointer named
 * *_host is host memory and *_dev is memory of the CUDA device the handle was
 * packed for.
 */
#ifndef XGEN_PATCONV_H
#define XGEN_PATCONV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct xgen_patconv_packed xgen_patconv_packed; /* opaque; owns host and device memory */

typedef enum {
    XGEN_OK = 0,
    XGEN_ERR_INVALID_ARG = 1,  /* null pointer, misaligned pointer, non-positive size          */
    XGEN_ERR_BAD_PATTERN = 2,  /* mask without exactly 4 of 9 bits, or pattern id out of range  */
    XGEN_ERR_SHAPE = 3,        /* tensor extents that do not fit the packed layer or 32-bit indexing */
    XGEN_ERR_UNSUPPORTED = 4,  /* stride, padding or data type outside what is built            */
    XGEN_ERR_ALLOC = 5,        /* host or device allocation failed                               */
    XGEN_ERR_CUDA = 6,         /* a CUDA runtime call failed, or the handle has no device copy   */
    XGEN_ERR_TIMEOUT = 7       /* a device-side bounded wait ran out (see xgen_patconv_last_status) */
} xgen_status;

/* Numeric variants.  F32: x, W, y fp32.  F16_F32ACC: x, W, y IEEE fp16, bias
 * fp32, sums and bias+ReLU in fp32, one round-to-nearest-even at the store.
 * I8_I32: x uint8 (zero point 0), W int8, bias int32, y int32 (the exact
 * integer sum, before any requantisation; scales are the caller's metadata). */
typedef enum { XGEN_F32 = 0, XGEN_F16_F32ACC = 1, XGEN_I8_I32 = 2 } xgen_dtype;

typedef struct {
    int32_t c_in;                   /* input channels,  >= 1                                   */
    int32_t c_out;                  /* output channels (filters), >= 1                         */
    int32_t stride;                 /* 1 or 2                                                  */
    int32_t pad;                    /* must be 1                                               */
    xgen_dtype dtype;
    int32_t num_patterns;           /* P, 1..126                                               */
    const uint16_t *pattern_masks;  /* [P] host; bit (3*dy+dx) set = tap kept; popcount 4      */
} xgen_patconv_desc;

/* What xgen_patconv_query reports about a packed layer. */
typedef struct {
    int64_t kernels_total;        /* c_in * c_out                                             */
    int64_t kernels_surviving;    /* kernels with a pattern (not removed)                     */
    int64_t macs_per_pixel;       /* 4 * kernels_surviving: useful multiply-adds per output pixel */
    int64_t weight_bytes;         /* bytes of kept weights at the layer's storage precision   */
    int64_t index_bytes;          /* bytes the device copy stores beyond weight_bytes: the
                                     command stream (48-byte slots: 16 bytes of opcode and
                                     operand, every kept weight widened to fp32 and stored
                                     twice) plus the offset and slot tables, less weight_bytes */
    int64_t compact_index_bytes;  /* the information in those bytes: one opcode byte and one
                                     operand byte per command, plus the offset and slot tables
                                     (what a byte-packed encoding of this layout would take)   */
    int64_t csr_index_bytes;      /* index bytes CSR would need for the same non-zeros
                                     (one 4-byte column per weight + one row pointer per filter) */
    int64_t stream_bytes;         /* bytes of the command stream as stored on the device
                                     (48-byte slots: every kept weight is stored twice there) */
    int32_t filters_per_group;    /* J: filters one warp accumulates together                 */
    int32_t groups_per_block;     /* filter groups (warps) per thread block                   */
    int32_t n_blocks;             /* blocks of contiguous output channels                     */
    int32_t channels_per_chunk;   /* input channels staged per pipeline step                  */
    int32_t n_chunks;
    int32_t patterns_compiled;    /* size of the compiled pattern table the layer runs with   */
    int32_t max_segment_slots;    /* longest per-(block, chunk) command segment               */
    int64_t load_commands;        /* activation-patch loads in the stream (one per group and
                                     input channel that group is connected to)                */
    double  group_imbalance;      /* worst thread block: max / mean of surviving kernels over
                                     the block's groups (its warps share the staged tiles)    */
} xgen_patconv_stats;

/* Read-only view of the packed layout on the host, for inspection and tests.
 * All pointers belong to the handle.
 *
 * The stream is an array of 32-byte command slots (8 words):
 *   word 0  opcode:  p < patterns_compiled  -> kernel command with compiled pattern p
 *                    patterns_compiled      -> LOAD: fetch the activation patch of one channel
 *                    patterns_compiled + 1  -> END of this group's commands for the chunk
 *   word 1  operand: kernel command: T * j (j = filter slot inside the group; T = 16 at
 *                    stride 1, 8 at stride 2: the output pixels one thread owns);
 *                    LOAD: channel index inside the chunk
 *   word 4..7  kernel command: the four kept weights in ascending tap order, fp32 bit
 *              patterns (fp16 and int8 weights are widened exactly)
 * Slots are ordered [block][chunk][group]: seg_off[(b * n_chunks + c) * (G + 1) + g]
 * (G = groups_per_block) is the first slot of group g of block b in chunk c, and
 * entry g = G is one past the segment.  Inside a group's run every LOAD is
 * followed by the kernel commands of that channel, and the run ends with END.
 * slot_oc[(b * G + g) * J + j] is the original output channel of filter slot j,
 * or -1 for an empty slot.
 * The device copy holds the same commands as 48-byte slots
 * {opcode, operand, -, -, w0, w0, w1, w1, w2, w2, w3, w3}. */
typedef struct {
    const uint32_t *slots;          int64_t n_slots;
    const int32_t  *seg_off;        /* [n_blocks * n_chunks * (G + 1)]                         */
    const int32_t  *slot_oc;        /* [n_blocks * G * J]                                      */
    const uint16_t *compiled_masks; /* [patterns_compiled]                                     */
} xgen_patconv_host_view;

/*
 * Pack one layer (paper Sec. 2.3, "Filter Kernel Reorder and Compact FKW
 * Storage": patterns are known after training, so filters are regrouped and
 * each filter's kernels reordered offline, and the weights are stored with one
 * index per kernel rather than per weight).
 *   dense_w_host    [c_out][c_in][3][3]: fp32 (XGEN_F32), IEEE fp16 bits
 *                   (XGEN_F16_F32ACC) or int8 (XGEN_I8_I32).  Values at pruned
 *                   positions are ignored; they need not be zero.
 *   pattern_id_host [c_out][c_in]: index into desc->pattern_masks, or -1 for a
 *                   removed kernel.
 *   device          CUDA device ordinal to upload to, or -1 to build the host
 *                   layout only (no CUDA call is made; such a handle cannot run).
 *   out             receives the handle; release it with xgen_patconv_free.
 * Synchronous.  Inputs are copied; the caller may free them on return.
 * Errors: INVALID_ARG, BAD_PATTERN, UNSUPPORTED (pad != 1, stride not 1|2),
 * SHAPE, ALLOC, CUDA.
 */
xgen_status xgen_patconv_pack(const xgen_patconv_desc *desc, const void *dense_w_host,
                              const int16_t *pattern_id_host, int device,
                              xgen_patconv_packed **out);

/*
 * Run the layer (paper Sec. 2.3, "Load Redundancy Elimination": tiled input,
 * per-pattern code with static tap offsets; Sec. 2.2: bias and ReLU fused).
 *   x_dev    [n][h][w][c_in]  NHWC, dtype's activation type, 16-byte aligned
 *   bias_dev [c_out] fp32 (int32 for XGEN_I8_I32), 4-byte aligned, or NULL for no bias
 *   relu     non-zero applies max(.,0)
 *   y_dev    [n][ho][wo][c_out] NHWC, 16-byte aligned, must not overlap x_dev;
 *            ho, wo as xgen_patconv_out_shape reports
 *   cuda_stream  a cudaStream_t passed as void* (NULL = default stream)
 * Only enqueues work on the stream: no synchronisation, no device allocation.
 * The caller keeps x, bias and y alive until the stream reaches that work.
 * Concurrent calls on different streams are allowed for unplanned shapes (the
 * handle only remembers, under a lock, the launch geometry and tensor map of the
 * last few (shape, x address) pairs, so repeated calls skip that work).  For a
 * shape prepared with xgen_patconv_plan see the rules there.
 * Errors: INVALID_ARG (null or misaligned pointer, y overlapping x), SHAPE
 * (n,h,w < 1 or a tensor beyond 2^31-1 elements), UNSUPPORTED (a tile of this
 * shape does not fit shared or tensor memory), CUDA (launch failure or
 * host-only handle).
 */
xgen_status xgen_patconv_run(const xgen_patconv_packed *packed, const void *x_dev, int32_t n,
                             int32_t h, int32_t w, const void *bias_dev, int32_t relu,
                             void *y_dev, void *cuda_stream);

/*
 * The operators that may be fused behind the convolution (paper Sec. 2.2, "universal
 * operator fusion": operators that follow a convolution are computed with it, so the
 * intermediate results never travel to memory and back).  With v the convolution's result
 * including the bias, in this order:
 *   residual_dev       NULL, or a tensor shaped like the convolution's own output
 *                      [n][ho][wo][c_out] in the output's element type (fp32, fp16, int32),
 *                      16-byte aligned: v += residual (the shortcut of a residual block)
 *   relu               non-zero: v = max(v, 0)
 *   pool               0, or 2: a 2x2 max-pool of stride 2 (VGG's stage ends); ho and wo must
 *                      be even, the stored result is [n][ho/2][wo/2][c_out]
 *   requant_scale_dev  XGEN_I8_I32 only: NULL (int32 result), or [c_out] fp32 scales, 4-byte
 *                      aligned: the result is stored as uint8 codes
 *                      clamp(rne(float(v) * scale[oc]) + requant_zero_point, 0, 255), where
 *                      float(v) is the int32 value rounded to fp32, the product is one fp32
 *                      multiplication and rne rounds to the nearest integer, ties to even
 */
typedef struct {
    int32_t relu;
    int32_t pool;
    const void *residual_dev;
    const float *requant_scale_dev;
    int32_t requant_zero_point;
} xgen_patconv_epilogue;

/*
 * xgen_patconv_run with the fused operators of *epilogue behind the convolution; `relu` of
 * xgen_patconv_run is epilogue->relu here.  y_dev holds the stored result as described above
 * (16-byte aligned; must overlap neither x_dev nor residual_dev).  Planned shapes (splits)
 * are honoured as in xgen_patconv_run.
 * Errors as xgen_patconv_run, plus INVALID_ARG (NULL epilogue, misaligned residual or scale),
 * SHAPE (pooling an odd extent), UNSUPPORTED (pool other than 0 or 2; re-quantisation of a
 * floating-point layer; a handle whose last xgen_patconv_plan chose 4x2-pixel blocks -- plan
 * it again with xgen_patconv_tuning.no_small_blocks).
 */
xgen_status xgen_patconv_run_fused(const xgen_patconv_packed *packed, const void *x_dev, int32_t n,
                                   int32_t h, int32_t w, const void *bias_dev,
                                   const xgen_patconv_epilogue *epilogue, void *y_dev,
                                   void *cuda_stream);

/*
 * (The paper has no counterpart to this entry point; it exists for callers of this
 * library.)  Run the layer with its input channels split over `splits` groups of thread
 * blocks, like a shape prepared with xgen_patconv_plan, but keep the partial sums in a
 * fixed array inside the library instead of a workspace from cudaMalloc.  It is meant for
 * callers that must not allocate device memory where they call us: code running under a
 * memory budget that was handed out up front, inside another framework's allocator
 * scope, or on a path where an allocation (which may synchronise the device) is not
 * allowed.  Neither this call nor anything it uses allocates or frees device memory.
 *
 *   splits   how many ways to split the channel chunks (>= 1; clamped to the number of
 *            chunks); more splits put more thread blocks to work on layers with few
 *            output pixels, and cost splits x 4 bytes of scratch per output element
 *   others   exactly as xgen_patconv_run; the caller still owns x, bias and y
 *
 * Limit: s x n*ho*wo*c_out x 4 bytes must not exceed
 * XGEN_PATCONV_STATIC_SCRATCH_BYTES, where s is the number of splits that actually get
 * channel chunks (splits after clamping, rounded so that every split has the same
 * number of chunks; s = 1 needs no scratch); beyond that the call returns XGEN_ERR_SHAPE and
 * launches nothing (with XGEN_PATCONV_LOG set, the reason goes to stderr).  The array is
 * part of the loaded library: every GPU that uses the library holds those bytes until
 * the process exits.
 * The first call on a device looks up the array's device address (once per device, with
 * that device made current); make that first call outside any stream capture.
 * All calls share the one array and nothing in it has to start at zero: every element a
 * call reads it has written itself.  For the same reason two calls whose kernels may
 * overlap on the GPU (different streams, no dependency between them) race on it; put
 * such calls on one stream or order them with events.
 * Errors: INVALID_ARG, SHAPE, CUDA, as xgen_patconv_run, plus SHAPE for the limit.
 */
#define XGEN_PATCONV_STATIC_SCRATCH_BYTES (8u << 20)
xgen_status xgen_patconv_run_static_scratch(const xgen_patconv_packed *packed, const void *x_dev,
                                            int32_t n, int32_t h, int32_t w, const void *bias_dev,
                                            int32_t relu, void *y_dev, int32_t splits,
                                            void *cuda_stream);

/*
 * Convenience for callers that hold host tensors: copies x (and bias) to the
 * device, runs the layer on the default stream, copies y back and waits
 * (xgen_patconv_enqueue_host followed by the wait).  The
 * device staging buffers belong to the handle and are kept between calls (they
 * only grow); calls on one handle are serialised.  Pinned (page-locked) host
 * memory makes the copies faster but is not required.  Same tensor layouts as
 * xgen_patconv_run, all pointers host memory.  Errors as xgen_patconv_run, plus ALLOC.
 */
xgen_status xgen_patconv_run_host(const xgen_patconv_packed *packed, const void *x_host, int32_t n,
                                  int32_t h, int32_t w, const void *bias_host, int32_t relu,
                                  void *y_host);

/*
 * The same three steps, only enqueued, without waiting: x (and bias) are copied to the
 * handle's device staging buffers on a stream of the handle's own, the layer (Sec. 2.1,
 * Sec. 2.2, as xgen_patconv_run) runs on cuda_stream (NULL = the default stream) once they
 * are there, and y is copied back on a second stream of the handle's own.  The caller's
 * stream thus carries kernels only: with page-locked host memory the call returns at once
 * and a sequence of such calls on different handles overlaps the copies in, the kernels
 * and the copies out with each other, in one caller stream.  With pageable memory the
 * copies may block the caller.  x_host and bias_host must stay unchanged, and y_host is
 * undefined, until xgen_patconv_last_status(packed, cuda_stream) has returned: it waits
 * for the stream and for the handle's copies and reports a kernel whose bounded wait ran
 * out.  Work enqueued on cuda_stream after this call is NOT ordered after the copy of y.
 * A further host-buffer call on the same handle waits, on the device, until this one
 * has released the staging buffers.  A staging buffer that has to grow is reallocated,
 * which synchronises the device; streams and events are created at the first call.  Not
 * for use inside a stream capture.  Errors as xgen_patconv_run, plus ALLOC.
 */
xgen_status xgen_patconv_enqueue_host(const xgen_patconv_packed *packed, const void *x_host, int32_t n,
                                      int32_t h, int32_t w, const void *bias_host, int32_t relu,
                                      void *y_host, void *cuda_stream);

/*
 * Optional: prepare the handle for one input shape.  Layers with few output
 * pixels do not fill the GPU with (pixel tile x filter block) work items; for
 * such a shape this call lets later xgen_patconv_run calls split the input
 * channels across thread blocks (the paper does not discuss this; it is the
 * cross-channel reduction of this implementation).  Shapes with more items
 * than the GPU holds blocks run in waves; there the items of the last, partly
 * filled wave are split the same way, so that the wave ends sooner.  The blocks of a split write
 * their partial sums to a workspace and count themselves in, all inside the one
 * kernel; the planner then picks one of two ways to add the sums up (see
 * xgen_patconv_plan_stats.last_arriver).
 *   Waiting splits: the blocks wait (with a bound in time) for the others and each
 * reduce a share.  Because they wait for each other, the split count is chosen so
 * that every block of the launch is resident at once on an otherwise idle GPU.
 * Hence the rule: such a launch must not share the GPU with another waiting split
 * launch -- of this handle or of any other handle -- nor with any other kernel
 * that may keep its blocks from becoming resident; put such launches on one
 * stream or order them with events.  If the rule is broken the blocks may hold
 * each other's places; the waits then run out (default 2 s), the kernel ends,
 * its results are invalid, and xgen_patconv_last_status returns
 * XGEN_ERR_TIMEOUT (xgen_patconv_run has returned XGEN_OK long before: it only
 * enqueues).  Work that merely delays the blocks (a kernel running before them
 * on the same stream) is harmless.
 *   Last arriver: nobody waits; the block of an item that counts itself in last adds
 * up all of the item's sums.  Any number of splits and of blocks is allowed (the
 * blocks run in waves), and other kernels, waiting splits of other handles among
 * them, may share the GPU.  It measured slower than waiting splits on every shape
 * tried, so the planner takes it only on request (xgen_patconv_tuning.reduce_mode
 * = 2): the mode for callers that run planned layers on several streams at once.
 *   Either way two planned split launches of ONE handle must not run at the same
 * time (they share the workspace and the counters): one stream, or events.
 * The call allocates the workspace and the counters, owned by the handle, so it
 * synchronises the device and must not be called while the handle is in use.
 * Without this call every shape runs unsplit.
 * Errors: INVALID_ARG, SHAPE, UNSUPPORTED, ALLOC, CUDA.
 */
xgen_status xgen_patconv_plan(xgen_patconv_packed *packed, int32_t n, int32_t h, int32_t w);

/*
 * The tuning-decided parameters of a layer (paper Sec. 2.3: the Layerwise
 * Representation carries "tuning-decided parameters" next to the pattern
 * information).  xgen_patconv_plan chooses them itself; a caller that has
 * measured better ones passes them here.  Zero in every field = the library's
 * own choice.
 *   splits             channel splits of the planned shape (clamped to what is
 *                      resident at once and to the number of channel chunks)
 *   no_copy_engine     stage input tiles with plain loads instead of the tensor
 *                      copy engine (every later run of the handle)
 *   no_launch_overlap  launch without programmatic stream serialisation, i.e. a
 *                      run starts only when its predecessor in the stream has
 *                      ended (every later run of the handle)
 *   wait_limit_ms      bound of the device-side waits, milliseconds (default
 *                      2000, at most 60000)
 *   no_small_blocks    keep 4x4 output pixels per thread even for shapes that the
 *                      planner would run with 4x2 pixels per thread (a single small
 *                      image); xgen_patconv_run_fused needs the 4x4 blocks
 *   channels_per_chunk input channels staged per pipeline step: 4, 8 or 16 (the command
 *                      stream is rebuilt and uploaded again; halved automatically while a
 *                      block's commands of one chunk exceed their 24 KB stage)
 *   groups_per_block   filter groups (consumer warps) per thread block, 1..16, at most the
 *                      library's own choice: fewer groups make more, smaller blocks of
 *                      output channels, hence more work items and fewer channel splits
 *   reduce_mode        how split items are added up: 0 or 1 by waiting splits, 2 by the
 *                      last arriver (then `splits` is clamped to the number of channel
 *                      chunks only, not to what is resident at once)
 */
typedef struct {
    int32_t splits;
    int32_t no_copy_engine;
    int32_t no_launch_overlap;
    int32_t wait_limit_ms;
    int32_t no_small_blocks;
    int32_t reduce_mode;
    int32_t channels_per_chunk;
    int32_t groups_per_block;
} xgen_patconv_tuning;

/* xgen_patconv_plan with the caller's tuning (NULL = xgen_patconv_plan).  Errors as
 * xgen_patconv_plan, plus INVALID_ARG for a negative field. */
xgen_status xgen_patconv_plan_tuned(xgen_patconv_packed *packed, int32_t n, int32_t h, int32_t w,
                                    const xgen_patconv_tuning *tuning);

/* How a run of an n x h x w input would be launched with the handle as it stands. */
typedef struct {
    int32_t splits;             /* channel splits (1 = unsplit; > 1 only for the planned shape)   */
    int32_t chunks_per_split;
    int32_t tiles;              /* pixel tiles                                                     */
    int32_t filter_blocks;      /* blocks of output channels                                       */
    int32_t items;              /* tiles x filter_blocks                                           */
    int32_t whole_items;        /* items that run as one block; the other items, numbered last,
                                   run as `splits` blocks each                                     */
    int32_t blocks;             /* thread blocks of the launch: whole_items + (items - whole_items) x splits */
    int32_t threads_per_block;
    int32_t row_tiling;         /* 0: a tile is a box of lanes_x x lanes_y blocks of lanes_n images;
                                   1: a tile is 32 consecutive blocks of the row-by-row numbering
                                   of all images' blocks (lanes_x = blocks per image row)         */
    int32_t lanes_x, lanes_y, lanes_n;  /* how a warp's 32 lanes tile x, y and images             */
    int32_t pixels_per_lane;    /* output pixels one lane owns: 16 (4x4) at stride 1, or 8 (4x2)
                                   where the planner chose the small block; 8 (2x4) at stride 2    */
    int32_t stages;             /* pipeline stages of staged channel chunks                        */
    int32_t uses_copy_engine;   /* input tiles arrive through the tensor copy engine               */
    int64_t shared_bytes;       /* dynamic shared memory per block                                 */
    int64_t workspace_bytes;    /* partial-sum workspace of the planned split, 0 if unsplit        */
    double  covered;            /* output pixels / pixel slots of all tiles (lanes x pixels each)  */
    int32_t last_arriver;       /* split items are added up by the block that arrives last (nobody
                                   waits) rather than by all of their blocks after a wait         */
    int32_t reserved;
} xgen_patconv_plan_stats;

/* Fill *stats for the shape.  No CUDA work is enqueued.  Errors: INVALID_ARG, SHAPE, UNSUPPORTED. */
xgen_status xgen_patconv_plan_info(const xgen_patconv_packed *packed, int32_t n, int32_t h, int32_t w,
                                   xgen_patconv_plan_stats *stats);

/*
 * Testing aid, not for production use (the paper has no counterpart): make every later
 * planned launch of waiting splits of the handle wait for `extra` arrivals more than its own blocks
 * will ever deliver.  With extra > 0 the wait of every block runs out after the handle's
 * wait limit (xgen_patconv_tuning.wait_limit_ms), the kernel ends normally, and
 * xgen_patconv_last_status returns XGEN_ERR_TIMEOUT once; extra = 0 restores normal
 * operation.  This is how the tests exercise the bounded waits without hanging or
 * faulting the GPU.  Errors: INVALID_ARG.
 */
xgen_status xgen_patconv_test_expect_arrivals(xgen_patconv_packed *packed, int32_t extra);

/* Output extents for an h x w input: ho = (h + 2 - 3) / stride + 1, likewise wo. */
xgen_status xgen_patconv_out_shape(const xgen_patconv_packed *packed, int32_t h, int32_t w,
                                   int32_t *ho, int32_t *wo);

/* Fill *stats (see xgen_patconv_stats). */
xgen_status xgen_patconv_query(const xgen_patconv_packed *packed, xgen_patconv_stats *stats);

/* Fill *view with pointers into the handle's host copy of the packed layout. */
xgen_status xgen_patconv_view(const xgen_patconv_packed *packed, xgen_patconv_host_view *view);

/* Synchronise the stream (and the handle's own copy streams, if xgen_patconv_enqueue_host was
 * used on it) and report the first CUDA error seen, as a status (XGEN_OK, XGEN_ERR_CUDA).  The kernels contain no unbounded waits: a wait
 * (for a staged tile, a free stage, or the other blocks of a split) that runs out
 * of its bound marks the handle, the kernel still ends, and this call then returns
 * XGEN_ERR_TIMEOUT once (results are invalid; the split counters are reset).  The
 * waits are bounded in time: 2 s unless xgen_patconv_tuning.wait_limit_ms says otherwise. */
xgen_status xgen_patconv_last_status(const xgen_patconv_packed *packed, void *cuda_stream);

/* Release the handle and its device memory.  NULL is allowed. */
void xgen_patconv_free(xgen_patconv_packed *packed);

/* Static, human-readable name of a status code. */
const char *xgen_strerror(xgen_status status);

/*
 * Measurement aid (the paper has no counterpart): rates of the arithmetic pipes that bound
 * the convolution kernels, from register-only microbenchmarks at full occupancy, and the
 * cost of launching a kernel shaped like them.  Runs a few kernels of about a millisecond
 * on the device's default stream and waits for them.
 *   ffma_tflops       scalar fp32 fused multiply-add (2 flop each)
 *   ffma2_tflops      packed two-wide fp32 fused multiply-add (the instruction the kernels use)
 *   dp4a_tmacs        u8 x s8 four-way dot product into int32, in 10^12 multiply-adds per second
 *   launch_floor_us   microseconds per launch over 200 back-to-back launches of an empty kernel
 *                     with the convolution kernels' block size, shared-memory carve-out,
 *                     tensor-memory allocation and launch attribute (128 blocks)
 *   single_launch_us  one such launch, from the event before it to the event after it
 *   sm_count, sm_clock_mhz  as the device reports them (the clock is the rated maximum)
 * Errors: INVALID_ARG, ALLOC, CUDA.
 */
typedef struct {
    double ffma_tflops, ffma2_tflops, dp4a_tmacs, launch_floor_us, single_launch_us;
    int32_t sm_count, sm_clock_mhz;
} xgen_patconv_probe_result;
xgen_status xgen_patconv_probe(int device, xgen_patconv_probe_result *result);

/* Number of kernel launches this library has enqueued in this process. */
int64_t xgen_patconv_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* XGEN_PATCONV_H */
