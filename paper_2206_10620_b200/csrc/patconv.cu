// libpatconv: CUDA kernels (sm_100a) and the C ABI.
//
// One thread block = one tile of output pixels x one block of contiguous output
// channels (x one range of input-channel chunks when the layer is split).  It has
// up to 16 consumer warps and four producer warps.
//
// Each consumer warp owns a filter group (J filters); each of its lanes owns a 4x4
// block of output pixels (2x4 at stride 2; up to LN images side by side for small
// images).  The warp interprets its command stream (core_gen.inc): LOAD brings the
// thread's activation patch of one channel into registers once, and every
// surviving kernel of the group on that channel reuses it (the paper's load
// redundancy elimination, Sec. 2.3); the running sums live in tensor memory,
// addressed by filter slot.
//
// The producer warps stage, per chunk of input channels, the input tile with its
// halo: the tensor copy engine delivers the NHWC box (zero-filled outside the
// image) and the block's slice of the command stream, and the producers spread
// the box into per-channel planes laid out as the operand pairs the two-wide FMAs
// read.  Channel counts the copy engine cannot address are read with plain loads.
// Stages are handed over with mbarriers (full / empty), so warps never meet at a
// block-wide barrier inside the main loop and a slow warp only delays the stage
// it still reads.
//
// The epilogue adds bias, applies ReLU, converts and stores straight from tensor
// memory: a group is a run of consecutive output channels, so a thread writes 32
// contiguous bytes per pixel (operator fusion, Sec. 2.2).
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <utility>
#include <new>
#include <vector>

#include "core_gen.inc"
#include "patconv_internal.h"

namespace patconv {

constexpr int kSmemPerSM = 233472;     // 228 KB
constexpr int kSmemMaxDynamic = 232448 - 2048;  // 227 KB per block less static shared memory
constexpr int kMaxWarps = 16;          // consumer warps
constexpr int kProducerWarps = 4;      // staging warps on top of them
constexpr int kDevSlotWords = 12;      // device command slot: 48 bytes (weights duplicated)
constexpr int kMaxStages = 4;
constexpr int kRawStages = 2;
constexpr size_t kCmdStageBudget = 24 * 1024;   // bytes of commands per pipeline stage the packer aims for

struct KParams {
    const void *x; void *y; const void *bias;
    const uint32_t *slots; const int32_t *seg_off; const int32_t *slot_oc;
    int n, h, w, ho, wo, c_in, c_out;
    int relu;
    // operators fused behind the convolution (all optional)
    const void *residual;                // tensor shaped like the unpooled result, result's element type: added before the activation
    const float *rq_scale;               // integer variant: per-channel scale of the re-quantisation to uint8, or null
    int rq_zero;                         // its zero point
    int pool;                            // 0, or 2 = 2x2 max-pool of stride 2
    int po, pw;                          // extents of the stored result (ho, wo, halved when pooling)
    int J, wpc, cc, n_chunks;
    int rc;                              // channels per tile box (a multiple of cc)
    int lx_log, ly_log, ln_log;          // grid tiling: lanes along x, y and images: 2^.. each, product 32
    // Row tiling (rows != 0): the 4x4 (2x4) pixel blocks of all images are numbered row by row
    // (image, block row, block column) and a tile is 32 consecutive blocks, one per lane; the
    // block rows it touches are staged one "slot" each (full image width, own halo rows).
    int rows;
    int bxn, byn;                        // blocks per image row, block rows per image
    uint32_t mg_bxn, mg_byn;
    int blocks_total;                    // n * byn * bxn
    int n_slots;                         // staged slots per tile: images (grid tiling) or block rows (row tiling)
    int slot_bytes;                      // bytes one tensor copy delivers in row tiling (one slot)
    int tiles_x, tiles_y;
    int tin_w, tin_h;                    // staged tile extents, input pixels
    uint32_t mg_tiles_x, mg_tiles_y, mg_tin_w, mg_tin_h, mg_spb;   // division by these as a multiplication (div_by)
    int spb;                             // chunks per tile box, rc / cc
    int pitch, img_stride, half_stride, plane_stride;   // words
    int raw_stage_words, plane_stage_words, cmd_stage_words;
    int n_stages;                        // plane + command stages
    int raw_off_words, plane_off_words, cmd_off_words;
    int tab_off_words;                   // per staged pixel: its two destinations inside a plane
    int src_off_words;                   // per staged pixel: element index in x, or -1 (plain-load staging)
    int ptab_off_words;                  // output-pixel table (32 lanes x pixels per thread)
    int seg_off_words;                   // the block's copy of the segment offsets
    int mbar_off_words;                  // 8-byte mbarriers: full, commands, empty (per stage), raw (per raw stage)
    int tmem_cols, cols_per_warp;
    int flush_chunks;                    // i8: chunks between folds of the fp32 partial sums
    int vec_out;                         // widest aligned store of an 8-channel piece: 8 or 4 words, 0 = scalar
    int use_tma;                         // stage tiles with the tensor copy engine (aligned channel counts)
    int box_bytes;                       // bytes one tensor copy delivers (the whole box, padding included)
    int *status;                         // device word: set to 1 if a bounded wait ran out
    int fold;                            // i8: keep int32 totals in a second row and fold periodically
    // Block numbering of a launch (one-dimensional grid): blocks 0 .. whole_items-1 each run one whole
    // item (tile, filter block); the remaining items follow, each as n_splits blocks that take
    // chunks_per_split channel chunks each.  A launch without splits has whole_items = all items.
    int whole_items;
    uint32_t mg_splits, mg_tiles;        // division by n_splits and by the number of tiles
    int n_tiles;
    int chunks_per_split;                // chunks one block of a split item takes
    uint32_t *partial;                   // split runs reduced by a second kernel: [split][n*ho*wo*c_out] raw sums
    size_t out_elems;                    // n*ho*wo*c_out
    // Split runs reduced inside this kernel: every block writes its raw sums as rows of
    // 32 lanes x 8 channels, [item][split][row][lane][8], item = (tile, filter block); a
    // counter per item tells when all of its splits have arrived, and each of them then
    // reduces a share of the rows.
    uint32_t *ws;
    uint32_t *counters;
    uint32_t target;                     // counter value at which every split of an item has arrived
    int n_splits;
    int last_reduces;                    // nobody waits: the block that arrives last adds up the whole item
    uint32_t wait_us;                    // bound of every device-side wait, microseconds
};

// ---- small PTX wrappers -----------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void tmem_ld8(uint32_t ta, uint32_t (&r)[8]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(ta) : "memory");
}
__device__ __forceinline__ void tmem_ld4(uint32_t ta, uint32_t (&r)[4]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(ta) : "memory");
}
__device__ __forceinline__ void tmem_st8(uint32_t ta, const uint32_t (&r)[8]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 ::"r"(ta), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]) : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ void mbar_init(uint32_t mbar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(mbar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t mbar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(mbar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t mbar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(mbar), "r"(bytes) : "memory");
}

__device__ __forceinline__ uint64_t global_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Wait for an mbarrier phase with a bound in time (limit_us microseconds, plus a cap on the
// polls in case the timer stands still): on expiry the block-wide abort flag and the device
// status word are set and every later wait returns at once; the warps then leave their
// loops, so the kernel still runs to its end (releasing tensor memory) with results the
// host can tell are invalid.
__device__ __forceinline__ bool mbar_wait(uint32_t mbar, uint32_t parity, volatile int *abort_flag, int *status,
                                          uint32_t limit_us) {
    uint64_t t0 = 0;
    for (uint32_t it = 0; it < 40000000u; ++it) {
        uint32_t ok;
        asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n selp.u32 %0, 1, 0, p;\n}"
                     : "=r"(ok) : "r"(mbar), "r"(parity), "r"(2000u) : "memory");
        if (ok) return true;
        if (*abort_flag) return false;
        if ((it & 7u) == 7u) {
            const uint64_t t = global_ns();
            if (t0 == 0) t0 = t;
            else if (t - t0 > (uint64_t)limit_us * 1000ull) break;
        }
    }
    *abort_flag = 1;
    if (status) atomicExch(status, 1);
    return false;
}

template <int STRIDE, int NP, int BH>
__device__ __forceinline__ void run_commands(uint32_t sp, uint32_t base_a, uint32_t plane_bytes,
                                             uint32_t pitch_bytes, uint32_t tmem_base, uint32_t base_b) {
    if (STRIDE == 1 && BH == 2) {
        if (NP == 4) PATCONV_CORE_S1H2_NP4(sp, base_a, plane_bytes, pitch_bytes, tmem_base, base_b);
        else if (NP == 8) PATCONV_CORE_S1H2_NP8(sp, base_a, plane_bytes, pitch_bytes, tmem_base, base_b);
        else if (NP == 12) PATCONV_CORE_S1H2_NP12(sp, base_a, plane_bytes, pitch_bytes, tmem_base, base_b);
        else PATCONV_CORE_S1H2_NP126(sp, base_a, plane_bytes, pitch_bytes, tmem_base, base_b);
    } else if (STRIDE == 1) {
        if (NP == 4) PATCONV_CORE_S1_NP4(sp, base_a, plane_bytes, pitch_bytes, tmem_base, base_b);
        else if (NP == 8) PATCONV_CORE_S1_NP8(sp, base_a, plane_bytes, pitch_bytes, tmem_base, base_b);
        else if (NP == 12) PATCONV_CORE_S1_NP12(sp, base_a, plane_bytes, pitch_bytes, tmem_base, base_b);
        else PATCONV_CORE_S1_NP126(sp, base_a, plane_bytes, pitch_bytes, tmem_base, base_b);
    } else {
        if (NP == 4) PATCONV_CORE_S2_NP4(sp, base_a, plane_bytes, pitch_bytes, tmem_base, base_b);
        else if (NP == 8) PATCONV_CORE_S2_NP8(sp, base_a, plane_bytes, pitch_bytes, tmem_base, base_b);
        else if (NP == 12) PATCONV_CORE_S2_NP12(sp, base_a, plane_bytes, pitch_bytes, tmem_base, base_b);
        else PATCONV_CORE_S2_NP126(sp, base_a, plane_bytes, pitch_bytes, tmem_base, base_b);
    }
}

// Element sizes of the activations (in) and the results (out).
template <int DT> struct DTraits;
template <> struct DTraits<XGEN_F32> { static constexpr int xbytes = 4, ybytes = 4; };
template <> struct DTraits<XGEN_F16_F32ACC> { static constexpr int xbytes = 2, ybytes = 2; };
template <> struct DTraits<XGEN_I8_I32> { static constexpr int xbytes = 1, ybytes = 4; };

// One staged activation element widened to fp32 (exact for fp16 and for uint8).
template <int DT> __device__ __forceinline__ float load_widened(const char *p) {
    if (DT == XGEN_F32) return __ldg(reinterpret_cast<const float *>(p));
    if (DT == XGEN_F16_F32ACC) return __half2float(__ushort_as_half(__ldg(reinterpret_cast<const unsigned short *>(p))));
    return (float)__ldg(reinterpret_cast<const unsigned char *>(p));
}

// One piece of the result: 8 adjacent output channels of one pixel, as 32-bit values (fp32 bits, or
// int32 for the integer variant).

// Raw sums stored as they are (partial sums of a split run): element offset o of a 32-bit array.
__device__ __forceinline__ void store_raw_piece(const KParams &P, const uint32_t (&r)[8], uint32_t *out, size_t o, int nv) {
    uint32_t *dst = out + o;
    if (nv == 8 && P.vec_out == 8) {
        asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(dst), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]) : "memory");
    } else if (nv == 8 && P.vec_out == 4) {
        *reinterpret_cast<uint4 *>(dst) = make_uint4(r[0], r[1], r[2], r[3]);
        *reinterpret_cast<uint4 *>(dst + 4) = make_uint4(r[4], r[5], r[6], r[7]);
    } else {
#pragma unroll
        for (int k = 0; k < 8; ++k) if (k < nv) dst[k] = r[k];
    }
}

// Bias, the fused residual addition and the activation (operator fusion, Sec. 2.2), applied to the
// raw sums of the piece at channel oc0 of unpooled pixel pidx.
template <int DT, bool FUSED>
__device__ __forceinline__ void finish_piece(const KParams &P, const uint32_t (&raw)[8], const uint32_t (&bb)[8],
                                             int oc0, int nv, int pidx, uint32_t (&v)[8]) {
    uint32_t res[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    if (FUSED && P.residual) {
        const size_t o = (size_t)pidx * P.c_out + oc0;
        if (DT == XGEN_F16_F32ACC) {
            const __half *rp = (const __half *)P.residual + o;
            if (nv == 8 && P.vec_out >= 4 && (P.c_out & 7) == 0) {
                const uint4 q = __ldg(reinterpret_cast<const uint4 *>(rp));
                const uint32_t w4[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const __half2 hv = *reinterpret_cast<const __half2 *>(&w4[k]);
                    res[2 * k] = __float_as_uint(__low2float(hv)); res[2 * k + 1] = __float_as_uint(__high2float(hv));
                }
            } else {
#pragma unroll
                for (int k = 0; k < 8; ++k) if (k < nv) res[k] = __float_as_uint(__half2float(rp[k]));
            }
        } else {
            const uint32_t *rp = (const uint32_t *)P.residual + o;
            if (nv == 8 && P.vec_out >= 4) {
                const uint4 a = __ldg(reinterpret_cast<const uint4 *>(rp)), b = __ldg(reinterpret_cast<const uint4 *>(rp) + 1);
                res[0] = a.x; res[1] = a.y; res[2] = a.z; res[3] = a.w; res[4] = b.x; res[5] = b.y; res[6] = b.z; res[7] = b.w;
            } else {
#pragma unroll
                for (int k = 0; k < 8; ++k) if (k < nv) res[k] = __ldg(rp + k);
            }
        }
    }
    if (DT == XGEN_I8_I32) {
#pragma unroll
        for (int k = 0; k < 8; ++k) { int q = (int)raw[k] + (int)bb[k] + (int)res[k]; if (P.relu) q = max(q, 0); v[k] = (uint32_t)q; }
    } else {
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            float q = __fadd_rn(__uint_as_float(raw[k]), __uint_as_float(bb[k]));
            if (FUSED && P.residual) q = __fadd_rn(q, __uint_as_float(res[k]));
            if (P.relu) q = fmaxf(q, 0.f);
            v[k] = __float_as_uint(q);
        }
    }
}

// Element-wise maximum of two finished pieces (max-pool).
template <int DT>
__device__ __forceinline__ void max_piece(uint32_t (&a)[8], const uint32_t (&b)[8]) {
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        if (DT == XGEN_I8_I32) a[k] = (uint32_t)max((int)a[k], (int)b[k]);
        else a[k] = __float_as_uint(fmaxf(__uint_as_float(a[k]), __uint_as_float(b[k])));
    }
}

// Convert a finished piece to the result's element type and store it at element offset o of y:
// fp32 and int32 as they are, fp16 by one round-to-nearest-even, and the re-quantised integer
// result as uint8 codes clamp(rne(float(v) * scale) + zero point, 0, 255), decided in fp32.
// The re-quantised piece: codes clamp(rne(float(v) * scale) + zero point, 0, 255).  The rounding
// to the nearest integer (ties to even) and the clamps are the conversion instructions' own:
// float to int32 saturates, the zero point is added with saturation, int32 to uint8 saturates.
__device__ __forceinline__ void emit_requantised(const float (&sc)[8], int zero, unsigned char *dst, bool vec, int nv,
                                                 const uint32_t (&r)[8]) {
    uint32_t code[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const int q = __float2int_rn(__fmul_rn((float)(int)r[k], sc[k]));
        int qz;
        asm("add.sat.s32 %0, %1, %2;" : "=r"(qz) : "r"(q), "r"(zero));
        asm("cvt.sat.u8.s32 %0, %1;" : "=r"(code[k]) : "r"(qz));
    }
    if (vec) {
        uint2 pk;
        pk.x = code[0] | (code[1] << 8) | (code[2] << 16) | (code[3] << 24);
        pk.y = code[4] | (code[5] << 8) | (code[6] << 16) | (code[7] << 24);
        *reinterpret_cast<uint2 *>(dst) = pk;
    } else {
#pragma unroll
        for (int k = 0; k < 8; ++k) if (k < nv) dst[k] = (unsigned char)code[k];
    }
}

template <int DT, bool FUSED>
__device__ __forceinline__ void emit_piece(const KParams &P, const uint32_t (&r)[8], const float (&sc)[8], size_t o, int nv) {
    if (FUSED && DT == XGEN_I8_I32 && P.rq_scale) {
        emit_requantised(sc, P.rq_zero, (unsigned char *)P.y + o, nv == 8 && P.vec_out >= 4 && (P.c_out & 7) == 0, nv, r);
    } else if (DT != XGEN_F16_F32ACC) {
        store_raw_piece(P, r, (uint32_t *)P.y, o, nv);
    } else {
        __half *dst = (__half *)P.y + o;
        if (nv == 8 && P.vec_out >= 4 && (P.c_out & 7) == 0) {
            uint4 pk;
            __half2 h0 = __floats2half2_rn(__uint_as_float(r[0]), __uint_as_float(r[1]));
            __half2 h1 = __floats2half2_rn(__uint_as_float(r[2]), __uint_as_float(r[3]));
            __half2 h2 = __floats2half2_rn(__uint_as_float(r[4]), __uint_as_float(r[5]));
            __half2 h3 = __floats2half2_rn(__uint_as_float(r[6]), __uint_as_float(r[7]));
            pk.x = *reinterpret_cast<uint32_t *>(&h0); pk.y = *reinterpret_cast<uint32_t *>(&h1);
            pk.z = *reinterpret_cast<uint32_t *>(&h2); pk.w = *reinterpret_cast<uint32_t *>(&h3);
            *reinterpret_cast<uint4 *>(dst) = pk;
        } else {
#pragma unroll
            for (int k = 0; k < 8; ++k) if (k < nv) dst[k] = __float2half_rn(__uint_as_float(r[k]));
        }
    }
}

// The four running sums of a thread that one pooled pixel q covers: stride 1 keeps sum
// 4*py + 2*h + e for pixel (py, h + 2*e) of its 4x4 block, so pooled pixel (qy, qx) = q / 2, q % 2
// covers py in {2qy, 2qy+1}, h in {0, 1}, e = qx; stride 2 keeps sum 2*py + e of its 2x4 block.
template <int STRIDE>
__device__ __forceinline__ int pool_member(int q, int m) {
    if (STRIDE == 1) return 4 * (2 * (q >> 1) + (m >> 1)) + 2 * (m & 1) + (q & 1);
    return 4 * q + m;
}

// n / d for the small divisors of the launch geometry: m = 2^32 / d + 1 (0 stands for d = 1),
// exact while n * d < 2^32.
__device__ __forceinline__ int div_by(int n, uint32_t m) { return m ? (int)__umulhi((uint32_t)n, m) : n; }

// Where a lane works: the first output pixel of its block, its image, and the word offset of
// its patch origin inside a channel plane (half 0).
struct LaneSite { int on, oy0, ox0, off; bool valid; };

// Where a staged slot comes from: image and input coordinates of its first staged pixel.
struct SlotOrigin { int gn, gy0, gx0; bool used; };

// ---- the kernel -----------------------------------------------------------------
// FUSED: with the operators fused behind the convolution (residual addition, max-pool,
// re-quantisation); the plain instances carry none of that code.
// BH: rows of the pixel block a thread owns (4; 2 = the small 4x2 block of stride 1).
template <int DT, int STRIDE, int NP, bool FUSED, int BH = 4>
__global__ void __launch_bounds__((kMaxWarps + kProducerWarps) * 32)
patconv_kernel(const KParams P, const __grid_constant__ CUtensorMap tmap) {
    extern __shared__ __align__(128) uint32_t smem[];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    __shared__ int soc_s[kMaxWarps * 16];           // original output channel of every filter slot of this block
    constexpr int XB = DTraits<DT>::xbytes;
    constexpr int BW = STRIDE == 1 ? 4 : 2;           // output pixels per thread: BW x BH
    constexpr int T = BW * BH;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nthreads = blockDim.x;
    const bool producer = warp >= P.wpc;
    const int pw = warp - P.wpc;                     // producer warp number
    // block -> (item, split); item -> (tile, block of output channels)
    const int blk = (int)blockIdx.x;
    const bool split_item = blk >= P.whole_items;
    const int tail = blk - P.whole_items;
    const int item = split_item ? P.whole_items + div_by(tail, P.mg_splits) : blk;
    const int zsplit = split_item ? tail - (item - P.whole_items) * P.n_splits : 0;
    const int sitem = item - P.whole_items;          // number of the item among the split ones
    const int b = div_by(item, P.mg_tiles);          // block of output channels
    const int tile = item - b * P.n_tiles;
    // grid tiling: tile -> (tx, ty, first image)
    const int tile_r = div_by(tile, P.mg_tiles_x);
    const int tx = tile - tile_r * P.tiles_x;
    const int tn = div_by(tile_r, P.mg_tiles_y);
    const int ty = tile_r - tn * P.tiles_y;
    const int LX = P.rows ? P.bxn : (1 << P.lx_log), LY = 1 << P.ly_log;
    const int TW = BW * LX, TH = BH * LY;
    const int n0 = tn << P.ln_log;                   // first image of the tile
    // row tiling: the tile's blocks 32*tile .. 32*tile+31 lie in block rows g_first .. g_last
    const int g_first = div_by(tile * 32, P.mg_bxn);
    const int g_last = div_by(min(tile * 32 + 31, P.blocks_total - 1), P.mg_bxn);
    auto lane_site = [&](int l) {
        LaneSite r;
        if (P.rows) {
            const int bl = tile * 32 + l;
            const int g = div_by(bl, P.mg_bxn), bx = bl - g * P.bxn;
            const int n = div_by(g, P.mg_byn), by = g - n * P.byn;
            r.on = n; r.oy0 = by * BH; r.ox0 = bx * BW;
            r.valid = bl < P.blocks_total;
            r.off = r.valid ? (g - g_first) * P.img_stride + bx * 4 : 0;   // idle lanes read slot 0
        } else {
            const int l_x = l & (LX - 1), l_y = (l >> P.lx_log) & (LY - 1), l_n = l >> (P.lx_log + P.ly_log);
            r.on = n0 + l_n; r.oy0 = ty * TH + l_y * BH; r.ox0 = tx * TW + l_x * BW;
            r.off = l_n * P.img_stride + l_y * BH * STRIDE * P.pitch + l_x * 4;
            r.valid = true;
        }
        return r;
    };
    auto slot_origin = [&](int sl) {
        SlotOrigin r;
        if (P.rows) {
            const int g = g_first + sl;
            const int n = div_by(g, P.mg_byn), by = g - n * P.byn;
            r.gn = n; r.gy0 = by * BH * STRIDE - 1; r.gx0 = -1; r.used = g <= g_last;
        } else {
            r.gn = n0 + sl; r.gy0 = ty * TH * STRIDE - 1; r.gx0 = tx * TW * STRIDE - 1; r.used = true;
        }
        return r;
    };
    const int slots_used = P.rows ? g_last - g_first + 1 : P.n_slots;
    const int NS = P.n_stages;
    const int npix = P.tin_w * P.tin_h * slots_used;       // staged pixels that are read
    const int npix_tab = P.tin_w * P.tin_h * P.n_slots;    // entries of the per-pixel tables

    const uint32_t smem_base = smem_u32(smem);
    const uint32_t mbar0 = smem_base + (uint32_t)P.mbar_off_words * 4u;
    auto bar_full = [&](int s) { return mbar0 + 8u * (uint32_t)s; };            // planes of a stage written
    auto bar_cmd = [&](int s) { return mbar0 + 8u * (uint32_t)(NS + s); };      // commands of a stage landed
    auto bar_empty = [&](int s) { return mbar0 + 8u * (uint32_t)(2 * NS + s); };   // every consumer warp done with a stage
    auto bar_raw = [&](int r) { return mbar0 + 8u * (uint32_t)(3 * NS + r); };  // a tile box landed
    auto bar_rawfree = [&](int r) { return mbar0 + 8u * (uint32_t)(3 * NS + kRawStages + r); };   // every producer warp done with a box

    const int c_begin = split_item ? zsplit * P.chunks_per_split : 0;
    const int c_end = split_item ? min(P.n_chunks, c_begin + P.chunks_per_split) : P.n_chunks;
    uint32_t *const ws_rows = split_item ? P.ws : nullptr;       // rows of partial sums exchanged inside the kernel
    uint32_t *const part_sums = split_item ? P.partial : nullptr; // or partial sums left to a second kernel

    // Launched with programmatic stream serialisation: the next kernel of the stream may be
    // scheduled as soon as SMs free up (its launch latency then overlaps this kernel's tail);
    // every kernel waits for its predecessors below, before it touches global memory.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    // --- tensor memory for the running sums; barriers -------------------------------
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_base_s)), "r"((uint32_t)P.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (pw == 0 && lane == 0) {
        abort_s = 0;
        for (int s = 0; s < NS; ++s) { mbar_init(bar_full(s), kProducerWarps); mbar_init(bar_cmd(s), 1); mbar_init(bar_empty(s), (uint32_t)P.wpc); }
        for (int r = 0; r < kRawStages; ++r) { mbar_init(bar_raw(r), 1); mbar_init(bar_rawfree(r), kProducerWarps); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();

    // From here on only the packed layer (commands, tables: written at pack time, before any
    // launch) is read without more ado.  Whatever an earlier kernel of the stream may have
    // produced or may still read -- x, y, the split's workspace and counters -- is touched only
    // after griddepcontrol.wait, by each thread that touches it: the table building below can
    // overlap the tail of the previous kernel.

    // A tile box carries rc channels, i.e. spb = rc / cc consecutive chunks; boxes q0..q_end
    // cover this block's chunks.  Box q is handed to the copy engine by one thread.
    const int spb = P.spb;
    const int q0 = div_by(c_begin, P.mg_spb), q_end = div_by(c_end - 1, P.mg_spb);
    auto issue_box = [&](int q) {
        const int r = (q - q0) % kRawStages;
        const uint32_t dst = smem_base + (uint32_t)(P.raw_off_words + r * P.raw_stage_words) * 4u;
        if (P.rows) {
            // one copy per block row the tile touches: full image width, own halo rows
            mbar_expect_tx(bar_raw(r), (uint32_t)(P.slot_bytes * slots_used));
            for (int sl = 0; sl < slots_used; ++sl) {
                const SlotOrigin o = slot_origin(sl);
                asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
                             ::"r"(dst + (uint32_t)(sl * P.slot_bytes)), "l"(&tmap), "r"(q * P.rc), "r"(o.gx0), "r"(o.gy0), "r"(o.gn), "r"(bar_raw(r)) : "memory");
            }
        } else {
            const SlotOrigin o = slot_origin(0);
            mbar_expect_tx(bar_raw(r), (uint32_t)P.box_bytes);
            asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
                         ::"r"(dst), "l"(&tmap), "r"(q * P.rc), "r"(o.gx0), "r"(o.gy0), "r"(o.gn), "r"(bar_raw(r)) : "memory");
        }
    };
    if (pw == 0 && lane == 0 && P.use_tma) {
        asm volatile("griddepcontrol.wait;" ::: "memory");       // x is complete
        for (int r = 0; r < kRawStages && q0 + r <= q_end; ++r) issue_box(q0 + r);
    }
    // The block's commands of chunk c (one contiguous segment [s0, s1) plus two look-ahead
    // slots), handed to the copy engine (one thread) for stage s.
    auto issue_commands = [&](int s, int s0, int s1) {
        const uint32_t cmd_bytes = (uint32_t)(s1 - s0 + 2) * (kDevSlotWords * 4u);
        const uint32_t cmd = smem_base + (uint32_t)(P.cmd_off_words + s * P.cmd_stage_words) * 4u;
        mbar_expect_tx(bar_cmd(s), cmd_bytes);
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(cmd), "l"(P.slots + (size_t)s0 * kDevSlotWords), "r"(cmd_bytes), "r"(bar_cmd(s)) : "memory");
    };
    const int32_t *seg_g = P.seg_off + ((size_t)b * P.n_chunks + c_begin) * (P.wpc + 1);
    // The first stages are free: their commands start now, with offsets read straight from
    // global memory, instead of after the tables below are built.
    if (pw == 0 && lane == 0)
        for (int k = 0; k < NS && c_begin + k < c_end; ++k)
            issue_commands(k, __ldg(seg_g + k * (P.wpc + 1)), __ldg(seg_g + k * (P.wpc + 1) + P.wpc));
    // Global reads of the tables below, started before the index arithmetic they do not need.
    const int soc_v = tid < P.wpc * P.J ? __ldg(P.slot_oc + (size_t)b * P.wpc * P.J + tid) : -1;
    const int n_seg = (c_end - c_begin) * (P.wpc + 1);
    const int seg_v = tid < n_seg ? __ldg(seg_g + tid) : 0;

    // --- tables, built once by all threads while the first boxes are in flight --------
    // Per staged pixel: where its value goes inside a channel plane.  A plane holds, per
    // tile row and lane column, half 0 = input columns (0,2,1,3) of that lane's patch and
    // half 1 = (2,4,3,5) (stride 2: (2,4)): the operand pairs of the two-wide FMAs.  A
    // pixel therefore lands in at most two places.
    int2 *tab = reinterpret_cast<int2 *>(smem + P.tab_off_words);
    int *srct = reinterpret_cast<int *>(smem + P.src_off_words);
    for (int q = tid; q < npix_tab; q += nthreads) {
        const int t2 = div_by(q, P.mg_tin_w), col = q - t2 * P.tin_w;
        const int im = div_by(t2, P.mg_tin_h), row = t2 - im * P.tin_h;
        const int base = im * P.img_stride + row * P.pitch;
        const int bx = col >> 2, cq = col & 3;
        int d0 = -1, d1 = -1;
        auto put = [&](int half, int word, int bxx) {
            const int o = half * P.half_stride + base + bxx * 4 + word;
            if (d0 < 0) d0 = o; else d1 = o;
        };
        if (bx < LX) {
            if (cq == 0) put(0, 0, bx);
            else if (cq == 1) put(0, 2, bx);
            else if (cq == 2) { put(0, 1, bx); put(1, 0, bx); }
            else { put(0, 3, bx); if (STRIDE == 1) put(1, 2, bx); }
        }
        if (bx >= 1 && bx - 1 < LX) {
            if (cq == 0) put(1, 1, bx - 1);
            else if (cq == 1 && STRIDE == 1) put(1, 3, bx - 1);
        }
        tab[q] = make_int2(d0, d1);
        if (!P.use_tma) {
            const SlotOrigin o = slot_origin(im);
            const int gy = o.gy0 + row, gx = o.gx0 + col, gn = o.gn;
            const bool ok = o.used && gn < P.n && gy >= 0 && gy < P.h && gx >= 0 && gx < P.w;
            srct[q] = ok ? ((gn * P.h + gy) * P.w + gx) * P.c_in : -1;
        }
    }
    // The staging warps need the table above and nothing of what follows: they wait for it
    // here (named barrier 1, every thread of the block counted once) and start on the first
    // tile, while the consumer warps only announce their entries and go on with their own tables.
    if (producer) asm volatile("bar.sync 1, %0;" ::"r"(nthreads) : "memory");
    else { __threadfence_block(); asm volatile("bar.arrive 1, %0;" ::"r"(nthreads) : "memory"); }
    const int cthreads = P.wpc * 32;
    if (tid < P.wpc * P.J) soc_s[tid] = soc_v;                       // wpc * J <= consumer threads
    // Output-pixel table: linear pixel index of (sum t of lane l), or -1 outside the output.
    // Stride 1 keeps a row's four pixels as the pairs (0,2) and (1,3): sum 4*py + 2*h + e is
    // pixel (py, h + 2*e); stride 2: sum 2*py + e is pixel (py, e).
    int *ptab = reinterpret_cast<int *>(smem + P.ptab_off_words);
    for (int i = tid; !producer && i < 32 * T; i += cthreads) {
        const int t = i >> 5, l2 = i & 31;
        const LaneSite ls = lane_site(l2);
        const int py = STRIDE == 1 ? (t >> 2) : (t >> 1);
        const int px = STRIDE == 1 ? (((t >> 1) & 1) + 2 * (t & 1)) : (t & 1);
        const int ox = ls.ox0 + px, oy = ls.oy0 + py, on = ls.on;
        ptab[i] = (ls.valid && on < P.n && oy < P.ho && ox < P.wo) ? (on * P.ho + oy) * P.wo + ox : -1;
    }
    // With the fused 2x2 max-pool: linear index of pooled pixel q of lane l in the stored result
    // (its window lies inside the image or outside it as a whole: ho and wo are even).
    int *qtab = ptab + 32 * T;
    for (int i = tid; FUSED && !producer && P.pool && i < 32 * (T / 4); i += cthreads) {
        const int q = i >> 5, l2 = i & 31;
        const LaneSite ls = lane_site(l2);
        const int qy = STRIDE == 1 ? (q >> 1) : q, qx = STRIDE == 1 ? (q & 1) : 0;
        const int oy = ls.oy0 + 2 * qy, ox = ls.ox0 + 2 * qx;
        qtab[i] = (ls.valid && ls.on < P.n && oy < P.ho && ox < P.wo) ? (ls.on * P.po + (oy >> 1)) * P.pw + (ox >> 1) : -1;
    }
    // Segment offsets of this block's chunks.
    int *seg = reinterpret_cast<int *>(smem + P.seg_off_words);
    if (!producer) {
        if (tid < n_seg) seg[tid] = seg_v;
        for (int i = tid + cthreads; i < n_seg; i += cthreads) seg[i] = seg_g[i];
        // and clear their running sums
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t tw = tmem_base_s + (((uint32_t)(warp & 3) * 32u) << 16) + (uint32_t)((warp >> 2) * P.cols_per_warp);
        const uint32_t z[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        for (int c = 0; c < P.cols_per_warp; c += 8) tmem_st8(tw + c, z);
        tmem_wait_st();
        asm volatile("bar.sync 2, %0;" ::"r"(cthreads) : "memory");   // the consumer warps' tables are complete
    }
    const uint32_t tmem_cta = tmem_base_s;
    const uint32_t plane_bytes = (uint32_t)P.plane_stride * 4u, pitch_bytes = (uint32_t)P.pitch * 4u;

    if (producer) {
        // ===== producer warps: fill stage after stage; warp 0 also drives the copy engine =====
        asm volatile("griddepcontrol.wait;" ::: "memory");   // they read x themselves, or wait (with a bound) for its copies
        const int ptid = pw * 32 + lane;
        // Offsets of the next chunk's commands (the consumer warps' copy in shared memory may not
        // be written yet), fetched one chunk ahead by the thread that hands them to the copy engine.
        const bool cmd_thread = pw == 0 && lane == 0;
        int cmd_s0 = 0, cmd_s1 = 0;
        if (cmd_thread && c_begin + NS < c_end) { cmd_s0 = __ldg(seg_g + NS * (P.wpc + 1)); cmd_s1 = __ldg(seg_g + NS * (P.wpc + 1) + P.wpc); }
        // chunk k uses stage s = k mod NS in its round ph = (k / NS) mod 2
        for (int c = c_begin, s = 0, ph = 0; c < c_end; ++c, s = (s + 1 == NS ? 0 : s + 1), ph ^= (s == 0)) {
            const int k = c - c_begin;
            if (k >= NS && !mbar_wait(bar_empty(s), (uint32_t)(ph ^ 1), &abort_s, P.status, P.wait_us)) break;
            if (cmd_thread && k >= NS) {              // the first NS chunks' commands are on their way already
                issue_commands(s, cmd_s0, cmd_s1);
                if (c + 1 < c_end) { cmd_s0 = __ldg(seg_g + (k + 1) * (P.wpc + 1)); cmd_s1 = __ldg(seg_g + (k + 1) * (P.wpc + 1) + P.wpc); }
            }
            float *pl = reinterpret_cast<float *>(smem + P.plane_off_words + s * P.plane_stage_words);
            if (P.use_tma) {
                const int q = div_by(c, P.mg_spb), sub = c - q * spb;
                const int r = (q - q0) % kRawStages;
                if ((k == 0 || sub == 0) &&
                    !mbar_wait(bar_raw(r), (uint32_t)(((q - q0) / kRawStages) & 1), &abort_s, P.status, P.wait_us)) break;
                // the copy engine delivered [pixel][channel]; spread this chunk's channels into the
                // fp32 operand planes
                const int len = P.cc * XB, pix_bytes = P.rc * XB;          // bytes per pixel: chunk, box
                const char *rawb = reinterpret_cast<const char *>(smem + P.raw_off_words + r * P.raw_stage_words) + sub * len;
                const int ps = P.plane_stride;
#pragma unroll 2
                for (int i = ptid; i < npix; i += kProducerWarps * 32) {
                    const int2 d = tab[i];
                    if (d.x < 0) continue;                 // a padding column of a slot: no lane reads it
                    float *d0 = pl + d.x, *d1 = pl + (d.y >= 0 ? d.y : d.x);
                    const char *src = rawb + (size_t)i * pix_bytes;
                    auto word = [&](uint32_t w, int e) {                   // one 32-bit word = 4 / XB channels from e on
                        if (DT == XGEN_F32) {
                            const float v = __uint_as_float(w);
                            d0[e * ps] = v; d1[e * ps] = v;
                        } else if (DT == XGEN_F16_F32ACC) {
                            const __half2 hv = *reinterpret_cast<const __half2 *>(&w);
                            const float v0 = __low2float(hv), v1 = __high2float(hv);
                            d0[e * ps] = v0; d1[e * ps] = v0;
                            d0[(e + 1) * ps] = v1; d1[(e + 1) * ps] = v1;
                        } else {
#pragma unroll
                            for (int bq = 0; bq < 4; ++bq) {
                                const float v = (float)((w >> (8 * bq)) & 0xFFu);
                                d0[(e + bq) * ps] = v; d1[(e + bq) * ps] = v;
                            }
                        }
                    };
                    constexpr int EPW = 4 / XB;                            // channels per word
                    if (len >= 16) {
                        for (int h2 = 0; h2 < (len >> 4); ++h2) {
                            const uint4 wd = *reinterpret_cast<const uint4 *>(src + 16 * h2);
                            word(wd.x, (4 * h2) * EPW); word(wd.y, (4 * h2 + 1) * EPW);
                            word(wd.z, (4 * h2 + 2) * EPW); word(wd.w, (4 * h2 + 3) * EPW);
                        }
                    } else if (len == 8) {
                        const uint2 wd = *reinterpret_cast<const uint2 *>(src);
                        word(wd.x, 0); word(wd.y, EPW);
                    } else {
                        word(*reinterpret_cast<const uint32_t *>(src), 0);
                    }
                }
                __syncwarp();
                if ((sub == spb - 1 || c == c_end - 1) && q + kRawStages <= q_end) {
                    // the box is refilled once every producer warp has read its share of it
                    if (lane == 0) mbar_arrive(bar_rawfree(r));
                    if (pw == 0) {
                        if (!mbar_wait(bar_rawfree(r), (uint32_t)(((q - q0) / kRawStages) & 1), &abort_s, P.status, P.wait_us)) break;
                        if (lane == 0) {
                            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // reads of the box before its reuse
                            issue_box(q + kRawStages);
                        }
                    }
                }
            } else {
                // plain loads: any channel count, any alignment
                const char *xb = (const char *)P.x;
                const int ic0 = c * P.cc;
                for (int i = ptid; i < npix; i += kProducerWarps * 32) {
                    const int2 d = tab[i];
                    if (d.x < 0) continue;
                    const int src = srct[i];
                    float *d0 = pl + d.x, *d1 = pl + (d.y >= 0 ? d.y : d.x);
#pragma unroll 4
                    for (int e = 0; e < P.cc; ++e) {
                        const bool ok = src >= 0 && ic0 + e < P.c_in;
                        const float v = ok ? load_widened<DT>(xb + (size_t)(src + ic0 + e) * XB) : 0.f;
                        d0[e * P.plane_stride] = v; d1[e * P.plane_stride] = v;
                    }
                }
                __syncwarp();
            }
            if (lane == 0) mbar_arrive(bar_full(s));
        }
    } else {
        // ===== consumer warps ===========================================================
        const uint32_t tmem_warp = tmem_cta + (((uint32_t)(warp & 3) * 32u) << 16) + (uint32_t)((warp >> 2) * P.cols_per_warp);
        const uint32_t tmem_int = tmem_warp + (uint32_t)(P.J * T);   // i8 with folding: int32 totals

        // i8: fold the exact fp32 partial sums into the int32 totals and clear them
        auto fold_partial_sums = [&]() {
            for (int c8 = 0; c8 < P.J * T; c8 += 8) {
                uint32_t f[8], q[8];
                tmem_ld8(tmem_warp + c8, f);
                tmem_ld8(tmem_int + c8, q);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 8; ++i) { q[i] = (uint32_t)((int)q[i] + __float2int_rn(__uint_as_float(f[i]))); f[i] = 0u; }
                tmem_st8(tmem_int + c8, q);
                tmem_st8(tmem_warp + c8, f);
            }
            tmem_wait_st();
        };
        // i8 without folding (few channels): the fp32 sums are exact integers; convert in place
        auto sums_to_int = [&]() {
            for (int c8 = 0; c8 < P.J * T; c8 += 8) {
                uint32_t f[8];
                tmem_ld8(tmem_warp + c8, f);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 8; ++i) f[i] = (uint32_t)__float2int_rn(__uint_as_float(f[i]));
                tmem_st8(tmem_warp + c8, f);
            }
            tmem_wait_st();
        };

        const uint32_t thr_off = (uint32_t)lane_site(lane).off * 4u;
        const uint32_t half_bytes = (uint32_t)P.half_stride * 4u;

        // The first bounded wait below must not start counting while an earlier kernel of the
        // stream still runs (the copies it waits for are issued only after that kernel).
        asm volatile("griddepcontrol.wait;" ::: "memory");
        // --- main loop over channel chunks --------------------------------------------
        for (int c = c_begin, s = 0, ph = 0; c < c_end; ++c, s = (s + 1 == NS ? 0 : s + 1), ph ^= (s == 0)) {
            const int k = c - c_begin;
            const uint32_t par = (uint32_t)ph;
            if (!mbar_wait(bar_full(s), par, &abort_s, P.status, P.wait_us)) break;
            if (!mbar_wait(bar_cmd(s), par, &abort_s, P.status, P.wait_us)) break;
            const int s0 = seg[k * (P.wpc + 1)], sg = seg[k * (P.wpc + 1) + warp];
            const uint32_t sp = smem_base + (uint32_t)(P.cmd_off_words + s * P.cmd_stage_words) * 4u +
                                (uint32_t)(sg - s0) * (kDevSlotWords * 4u);
            const uint32_t base_a = smem_base + (uint32_t)(P.plane_off_words + s * P.plane_stage_words) * 4u + thr_off;
            run_commands<STRIDE, NP, BH>(sp, base_a, plane_bytes, pitch_bytes, tmem_warp, base_a + half_bytes);
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_empty(s));
            if (DT == XGEN_I8_I32 && P.fold && ((k + 1) % P.flush_chunks == 0)) fold_partial_sums();
        }
        if (DT == XGEN_I8_I32) { if (P.fold) fold_partial_sums(); else sums_to_int(); }

        // --- epilogue: bias + ReLU + convert, straight from tensor memory to NHWC -------
        // A group is a run of J consecutive output channels, so for one pixel a thread holds
        // 8 adjacent channels per 8 filter slots: 32 bytes (16 for fp16) it can store as one
        // piece.  No shared memory, no block-wide barrier: every warp drains on its own.
        asm volatile("griddepcontrol.wait;" ::: "memory");       // before the first store to y or the workspace
        const int *soc = soc_s + warp * P.J;
        const uint32_t tmem_res = (DT == XGEN_I8_I32 && P.fold) ? tmem_int : tmem_warp;
        const int oc_base = soc[0];
        if (oc_base >= 0) {
            uint32_t *const part = part_sums ? part_sums + (size_t)zsplit * P.out_elems : nullptr;
            const int K8 = (P.J + 7) >> 3;
            uint32_t *const wrow = ws_rows ? ws_rows + ((((size_t)sitem * P.n_splits + zsplit) * (size_t)(P.wpc * K8 * T)
                                                   + (size_t)warp * K8 * T) * 32 + lane) * 8 : nullptr;
            const int *pt = ptab + lane;
            const int *qtab = ptab + 32 * T;
            for (int j0 = 0; j0 < P.J; j0 += 8) {
                const int oc0 = oc_base + j0;
                if (oc0 >= P.c_out) break;
                const int nv = min(8, P.c_out - oc0);                 // valid channels of this piece
                uint32_t bb[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) bb[k] = (P.bias && !part && !wrow && k < nv) ? ((const uint32_t *)P.bias)[oc0 + k] : 0u;
                float sc[8];                                          // re-quantisation scales of these channels
#pragma unroll
                for (int k = 0; k < 8; ++k) sc[k] = (FUSED && DT == XGEN_I8_I32 && P.rq_scale && k < nv) ? __ldg(P.rq_scale + oc0 + k) : 0.f;
                if (FUSED && P.pool && !part && !wrow) {
                    // fused 2x2 max-pool: the four sums of a pooled pixel are columns of this thread
                    for (int q = 0; q < T / 4; ++q) {
                        const int qidx = qtab[q * 32 + lane];
                        uint32_t best[8], u[8], f[8];
                        for (int m = 0; m < 4; ++m) {
#pragma unroll
                            for (int k = 0; k < 8; ++k) {
                                if (j0 + k < P.J)
                                    asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];"
                                                 : "=r"(u[k]) : "r"(tmem_res + (j0 + k) * T + pool_member<STRIDE>(q, m)) : "memory");
                                else u[k] = 0u;
                            }
                            tmem_wait_ld();
                            if (qidx < 0) continue;
                            if (m == 0) finish_piece<DT, FUSED>(P, u, bb, oc0, nv, pt[pool_member<STRIDE>(q, 0) * 32], best);
                            else { finish_piece<DT, FUSED>(P, u, bb, oc0, nv, pt[pool_member<STRIDE>(q, m) * 32], f); max_piece<DT>(best, f); }
                        }
                        if (qidx < 0) continue;
                        emit_piece<DT, FUSED>(P, best, sc, (size_t)qidx * P.c_out + oc0, nv);
                    }
                    continue;
                }
                for (int t0 = 0; t0 < T; t0 += 4) {
                    uint32_t v[8][4];
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        if (j0 + k < P.J) tmem_ld4(tmem_res + (j0 + k) * T + t0, v[k]);
                        else { v[k][0] = v[k][1] = v[k][2] = v[k][3] = 0u; }
                    }
                    tmem_wait_ld();
#pragma unroll
                    for (int tt = 0; tt < 4; ++tt) {
                        uint32_t r[8];
#pragma unroll
                        for (int k = 0; k < 8; ++k) r[k] = v[k][tt];
                        if (wrow) {
                            // raw sums, one 1 KB row per warp and store: lanes side by side
                            uint32_t *dst = wrow + (size_t)(((j0 >> 3) * T + t0 + tt) * 32) * 8;
                            asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(dst), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]) : "memory");
                            continue;
                        }
                        const int pidx = pt[(t0 + tt) * 32];
                        if (pidx < 0) continue;
                        if (part) { store_raw_piece(P, r, part, (size_t)pidx * P.c_out + oc0, nv); continue; }
                        uint32_t f[8];
                        finish_piece<DT, FUSED>(P, r, bb, oc0, nv, pidx, f);
                        emit_piece<DT, FUSED>(P, f, sc, (size_t)pidx * P.c_out + oc0, nv);
                    }
                }
            }
        }
    }

    if (ws_rows) {
        // ===== split item: the partial sums of all splits of this item are added up either by
        // all of its blocks, each taking a share once every split has arrived (they wait for each
        // other: the planner keeps them within what the GPU holds at once), or, with any number
        // of splits, by whichever block arrives last (nobody waits) =====
        asm volatile("griddepcontrol.wait;" ::: "memory");       // the producer warps join in here
        __threadfence();
        __syncthreads();
        if (tid == 0 && P.last_reduces) {
            uint32_t old;
            asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(old) : "l"(P.counters + sitem) : "memory");
            if (old + 1u != P.target) abort_s = 2;                // not the last one: nothing left to do
        } else if (tid == 0) {
            uint32_t *cnt = P.counters + sitem;
            asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(cnt) : "memory");
            bool ok = false;
            uint64_t t0 = 0;
            for (uint32_t it = 0; it < 40000000u && !abort_s; ++it) {
                uint32_t v;
                asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(cnt) : "memory");
                if ((int)(v - P.target) >= 0) { ok = true; break; }
                __nanosleep(100);
                if ((it & 15u) == 15u) {
                    const uint64_t t = global_ns();
                    if (t0 == 0) t0 = t;
                    else if (t - t0 > (uint64_t)P.wait_us * 1000ull) break;
                }
            }
            if (!ok) { abort_s = 1; if (P.status) atomicExch(P.status, 1); }
        }
        __syncthreads();
        if (!abort_s) {
            const int K8 = (P.J + 7) >> 3;
            const int R = P.wpc * K8 * T, S = P.n_splits, nwarps = nthreads >> 5;
            const int row0 = P.last_reduces ? 0 : zsplit, rstep = P.last_reduces ? 1 : S;   // this block's share of the rows
            const uint32_t *base = ws_rows + (size_t)sitem * S * R * 256;
            const size_t zstride = (size_t)R * 64;                // uint4 per split
            // the sums of row `row` (one running sum of every lane, 8 channels) over all splits, in split order
            auto sum_row = [&](int row, uint32_t (&acc)[8]) {
#pragma unroll
                for (int k = 0; k < 8; ++k) acc[k] = 0u;
                auto add8 = [&](const uint4 &lo, const uint4 &hi) {
                    const uint32_t q[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        if (DT == XGEN_I8_I32) acc[k] = (uint32_t)((int)acc[k] + (int)q[k]);
                        else acc[k] = __float_as_uint(__uint_as_float(acc[k]) + __uint_as_float(q[k]));
                    }
                };
                const uint4 *src = reinterpret_cast<const uint4 *>(base + ((size_t)row * 32 + lane) * 8);
                for (int z = 0; z < S; z += 4) {                      // four splits in flight; summed in order 0, 1, ...
                    uint4 lo[4], hi[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        if (z + u < S) { lo[u] = __ldcg(src + (z + u) * zstride); hi[u] = __ldcg(src + (z + u) * zstride + 1); }
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        if (z + u < S) add8(lo[u], hi[u]);
                }
            };
            if (FUSED && P.pool) {
                // Units of one pooled pixel: (warp's filter group, 8-channel piece, pooled pixel q).  The
                // four running sums a unit covers are reduced by four warps side by side; they meet in
                // shared memory (the staging area is free by now), where the first of them takes the maximum.
                const int Q = T / 4, U = P.wpc * K8 * Q;
                const int *qtab = ptab + 32 * T;
                uint32_t *pool_s = smem + P.plane_off_words + (size_t)(warp * 32 + lane) * 8;
                const int per_pass = nwarps >> 2;
                for (int u0 = row0; u0 < U; u0 += rstep * per_pass) {
                    const int unit = u0 + rstep * (warp >> 2), m = warp & 3;
                    const bool mine = (warp >> 2) < per_pass && unit < U;
                    const int q = unit % Q, k8 = (unit / Q) % K8, w = unit / (Q * K8);
                    const int ocb = mine ? soc_s[w * P.J] : -1;
                    const int oc0 = ocb + k8 * 8;
                    const int qidx = mine ? qtab[q * 32 + lane] : -1;
                    const bool live = mine && ocb >= 0 && oc0 < P.c_out && qidx >= 0;
                    const int nv = min(8, P.c_out - oc0);
                    uint32_t bb[8], f[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k) bb[k] = (live && P.bias && k < nv) ? ((const uint32_t *)P.bias)[oc0 + k] : 0u;
                    if (live) {
                        uint32_t acc[8];
                        const int t = pool_member<STRIDE>(q, m);
                        sum_row((w * K8 + k8) * T + t, acc);
                        finish_piece<DT, FUSED>(P, acc, bb, oc0, nv, ptab[t * 32 + lane], f);
                        if (m != 0) {
                            *reinterpret_cast<uint4 *>(pool_s) = make_uint4(f[0], f[1], f[2], f[3]);
                            *reinterpret_cast<uint4 *>(pool_s + 4) = make_uint4(f[4], f[5], f[6], f[7]);
                        }
                    }
                    __syncthreads();
                    if (live && m == 0) {
                        for (int mm = 1; mm < 4; ++mm) {
                            const uint4 a = *reinterpret_cast<const uint4 *>(pool_s + (size_t)mm * 256);
                            const uint4 c = *reinterpret_cast<const uint4 *>(pool_s + (size_t)mm * 256 + 4);
                            const uint32_t g[8] = {a.x, a.y, a.z, a.w, c.x, c.y, c.z, c.w};
                            max_piece<DT>(f, g);
                        }
                        float sc[8];
#pragma unroll
                        for (int k = 0; k < 8; ++k) sc[k] = (DT == XGEN_I8_I32 && P.rq_scale && k < nv) ? __ldg(P.rq_scale + oc0 + k) : 0.f;
                        emit_piece<DT, FUSED>(P, f, sc, (size_t)qidx * P.c_out + oc0, nv);
                    }
                    __syncthreads();
                }
            } else {
                for (int row = row0 + rstep * warp; row < R; row += rstep * nwarps) {
                    const int t = row % T, k8 = (row / T) % K8, w = row / (T * K8);
                    const int ocb = soc_s[w * P.J];
                    const int oc0 = ocb + k8 * 8;
                    const int pidx = ptab[t * 32 + lane];
                    if (ocb < 0 || oc0 >= P.c_out || pidx < 0) continue;
                    const int nv = min(8, P.c_out - oc0);
                    uint32_t acc[8], f[8], bb[8];
                    sum_row(row, acc);
#pragma unroll
                    for (int k = 0; k < 8; ++k) bb[k] = (P.bias && k < nv) ? ((const uint32_t *)P.bias)[oc0 + k] : 0u;
                    float sc[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k) sc[k] = (FUSED && DT == XGEN_I8_I32 && P.rq_scale && k < nv) ? __ldg(P.rq_scale + oc0 + k) : 0.f;
                    finish_piece<DT, FUSED>(P, acc, bb, oc0, nv, pidx, f);
                    emit_piece<DT, FUSED>(P, f, sc, (size_t)pidx * P.c_out + oc0, nv);
                }
            }
        }
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_cta), "r"((uint32_t)P.tmem_cols) : "memory");
    }
}

// Split runs: y = act(bias + sum over splits of the raw partial sums), in a fixed
// order (split 0, 1, ...), four channels per thread.
template <int DT>
__global__ void __launch_bounds__(256)
patconv_reduce_kernel(const uint32_t *__restrict__ partial, int splits, size_t out_elems, int c_out,
                      const void *__restrict__ bias, int relu, void *__restrict__ y, int vec) {
    const size_t i = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * (vec ? 4 : 1);
    // Launched with programmatic stream serialisation: everything above overlaps the tail
    // of the convolution kernel; the partial sums are read only after it has completed.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (i >= out_elems) return;
    const int oc = (int)(i % (size_t)c_out);
    if (DT == XGEN_I8_I32) {
        int r[4] = {0, 0, 0, 0};
#pragma unroll 4
        for (int z = 0; z < splits; ++z) {
            const uint32_t *src = partial + (size_t)z * out_elems + i;
            if (vec) { const int4 v = *reinterpret_cast<const int4 *>(src); r[0] += v.x; r[1] += v.y; r[2] += v.z; r[3] += v.w; }
            else r[0] += (int)src[0];
        }
        for (int k = 0; k < (vec ? 4 : 1); ++k) {
            if (bias) r[k] += ((const int *)bias)[oc + k];
            if (relu) r[k] = max(r[k], 0);
            ((int *)y)[i + k] = r[k];
        }
    } else {
        float r[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 4
        for (int z = 0; z < splits; ++z) {
            const uint32_t *src = partial + (size_t)z * out_elems + i;
            if (vec) { const float4 v = *reinterpret_cast<const float4 *>(src); r[0] += v.x; r[1] += v.y; r[2] += v.z; r[3] += v.w; }
            else r[0] += __uint_as_float(src[0]);
        }
        for (int k = 0; k < (vec ? 4 : 1); ++k) {
            if (bias) r[k] += ((const float *)bias)[oc + k];
            if (relu) r[k] = fmaxf(r[k], 0.f);
        }
        if (DT == XGEN_F32) {
            if (vec) *reinterpret_cast<float4 *>((float *)y + i) = make_float4(r[0], r[1], r[2], r[3]);
            else ((float *)y)[i] = r[0];
        } else {
            if (vec) {
                __half2 lo = __floats2half2_rn(r[0], r[1]), hi = __floats2half2_rn(r[2], r[3]);
                uint2 pk;
                pk.x = *reinterpret_cast<uint32_t *>(&lo);
                pk.y = *reinterpret_cast<uint32_t *>(&hi);
                *reinterpret_cast<uint2 *>((__half *)y + i) = pk;
            } else ((__half *)y)[i] = __float2half_rn(r[0]);
        }
    }
}

// ---- host side ----------------------------------------------------------------------
static std::atomic<int64_t> g_launches{0};
void count_launch() { g_launches.fetch_add(1); }

// The one environment switch, read once when the library is first used.
static bool log_enabled() {
    static const bool on = getenv("XGEN_PATCONV_LOG") != nullptr;
    return on;
}

static inline int pixels_per_thread_x(int stride) { return stride == 1 ? 4 : 2; }

struct Geometry {
    int lx_log, ly_log, ln_log, tiles_x, tiles_y, tiles_n;
    int rows, bxn, byn, blocks_total, n_slots, tiles;   // row tiling (rows != 0); n_slots, tiles: either tiling
    int tin_w, tin_h, pitch, img_stride, half_stride, plane_stride;
    double covered;                                      // output pixels / pixel slots of all tiles
};

// Worst bank multiplicity of a thread's 128-bit patch-row load: `addr` gives the word offset of a
// lane's patch origin inside a plane; 128-bit accesses go out 8 lanes per wavefront.
template <typename F>
static int row_load_conflicts(F addr) {
    int worst = 0;
    for (int ph = 0; ph < 4; ++ph) {
        int cnt[32] = {0};
        for (int l = 0; l < 8; ++l) {
            int a = addr(ph * 8 + l);
            for (int k = 0; k < 4; ++k) cnt[(a + k) & 31]++;
        }
        for (int i = 0; i < 32; ++i) worst = worst > cnt[i] ? worst : cnt[i];
    }
    return worst;
}

// Grid tiling: the 32 lanes of a warp tile LX x LY x LN (powers of two) blocks of 4x4 (2x4)
// pixels; chosen to cover the most output pixels per tile.
static Geometry grid_geometry(int n, int ho, int wo, int stride, int bh) {
    Geometry best{};
    double best_eff = -1.0;
    const int bw = pixels_per_thread_x(stride);
    for (int lx_log = 5; lx_log >= 0; --lx_log)
        for (int ly_log = 5 - lx_log; ly_log >= 0; --ly_log) {
            const int ln_log = 5 - lx_log - ly_log;
            const int TW = bw << lx_log, TH = bh << ly_log, LN = 1 << ln_log;
            if (LN > 1 && (TW < wo || TH < ho)) continue;   // several images per tile only when one image fits
            const long tiles = (long)((wo + TW - 1) / TW) * ((ho + TH - 1) / TH) * ((n + LN - 1) / LN);
            const double eff = (double)n * ho * wo / ((double)tiles * 32.0 * bw * bh);
            if (eff > best_eff + 1e-9) {
                best_eff = eff;
                best.lx_log = lx_log; best.ly_log = ly_log; best.ln_log = ln_log;
            }
        }
    const int TW = bw << best.lx_log, TH = bh << best.ly_log, LN = 1 << best.ln_log;
    best.tiles_x = (wo + TW - 1) / TW; best.tiles_y = (ho + TH - 1) / TH; best.tiles_n = (n + LN - 1) / LN;
    best.tiles = best.tiles_x * best.tiles_y * best.tiles_n;
    best.n_slots = LN;
    best.blocks_total = 1 << 30;
    best.covered = best_eff;
    best.tin_w = stride == 1 ? TW + 2 : 2 * TW + 1;
    best.tin_h = stride == 1 ? TH + 2 : 2 * TH + 1;
    // One half of a plane row holds 4 words per lane column; pad the row and the image so
    // that the 128-bit loads of a quarter warp fall into distinct banks.
    const int p0 = 4 << best.lx_log;
    int best_p = p0, best_i = best.tin_h * p0, best_c = 1 << 30;
    for (int p = p0; p <= p0 + 12; p += 4)
        for (int ipad = 0; ipad <= (LN > 1 ? 28 : 0); ipad += 4) {
            const int istr = best.tin_h * p + ipad;
            const int LX = 1 << best.lx_log, LY = 1 << best.ly_log;
            const int c = row_load_conflicts([&](int lane) {
                int x = lane & (LX - 1), y = (lane >> best.lx_log) & (LY - 1), nn = lane >> (best.lx_log + best.ly_log);
                return nn * istr + y * bh * stride * p + x * 4;
            });
            if (c < best_c) { best_c = c; best_p = p; best_i = istr; }
        }
    best.pitch = best_p;
    best.img_stride = best_i;
    best.half_stride = LN * best.img_stride;
    best.plane_stride = 2 * best.half_stride;
    return best;
}

// Row tiling: the blocks of all images are numbered (image, block row, block column) and a
// tile takes 32 consecutive ones, so only the last tile of the launch has idle lanes; what is
// lost is the part of edge blocks that hangs over the image.  Every block row a tile touches is
// staged as a slot of its own: the full image width plus halo, with its own halo rows.
static bool row_geometry(int n, int ho, int wo, int stride, int bh, Geometry &g) {
    const int bw = pixels_per_thread_x(stride);
    const int bxn = (wo + bw - 1) / bw, byn = (ho + bh - 1) / bh;
    if (bxn > 32) return false;
    const int64_t total = (int64_t)n * byn * bxn;
    if (total > (int64_t)1 << 26) return false;
    g = Geometry{};
    g.rows = 1; g.bxn = bxn; g.byn = byn; g.blocks_total = (int)total;
    g.tiles = (int)((total + 31) / 32);
    g.tiles_x = g.tiles; g.tiles_y = 1; g.tiles_n = 1;
    g.n_slots = std::min<int64_t>((31 + bxn - 1) / bxn + 1, (int64_t)n * byn);   // most block rows 32 consecutive blocks touch
    g.covered = (double)n * ho * wo / ((double)g.tiles * 32.0 * bw * bh);
    g.tin_w = stride == 1 ? bxn * bw + 2 : 2 * bxn * bw + 1;
    g.tin_h = stride == 1 ? bh + 2 : 2 * bh + 1;
    // pad the row pitch and the slot stride so that a quarter warp's 128-bit loads spread over the banks,
    // whatever block column the tile starts at
    const int p0 = 4 * bxn;
    int best_p = p0, best_i = g.tin_h * p0, best_c = 1 << 30;
    for (int p = p0; p <= p0 + 12; p += 4)
        for (int ipad = 0; ipad <= 28; ipad += 4) {
            const int istr = g.tin_h * p + ipad;
            int c = 0;
            for (int start = 0; start < bxn; ++start)
                c = std::max(c, row_load_conflicts([&](int lane) {
                    const int bl = start + lane;
                    return (bl / bxn) * istr + (bl % bxn) * 4;
                }));
            if (c < best_c) { best_c = c; best_p = p; best_i = istr; }
        }
    g.pitch = best_p;
    g.img_stride = best_i;
    g.half_stride = g.n_slots * g.img_stride;
    g.plane_stride = 2 * g.half_stride;
    return true;
}

// Everything about a launch that depends only on the layer and the input shape: tile
// geometry, shared-memory layout, tensor-memory columns.
struct Layout {
    Geometry g;
    KParams kp;          // pointers, split and tensor-map fields left empty
    size_t smem;
    int items;           // (tile, filter block) pairs = blocks of an unsplit launch
};

// One prepared launch of a handle: the layout of a shape and the tensor map of an input
// address.  xgen_patconv_run looks its shape up here instead of redoing the geometry search
// and the tensor-map encoding on every call.
struct LaunchEntry {
    int n = 0, h = 0, w = 0;
    const void *x = nullptr;
    bool y32 = false;
    Layout L;
    CUtensorMap tm;
    uint64_t stamp = 0;
};
constexpr int kLaunchCache = 4;

}  // namespace patconv

using namespace patconv;

struct xgen_patconv_packed {
    PackedHost host;
    int device = -1;
    uint32_t *d_slots = nullptr;
    int32_t *d_seg_off = nullptr;
    int32_t *d_slot_oc = nullptr;
    // set by xgen_patconv_plan: split the channel chunks of this shape across blocks
    int plan_n = 0, plan_h = 0, plan_w = 0, plan_splits = 1, plan_cps = 0;
    int plan_whole = 0;                 // items of the planned shape that run whole (the others are split)
    bool plan_last = false;             // split items are added up by their last block to arrive (nobody waits)
    bool layout_asked = false;          // the current grouping was named by a caller's tuning
    uint32_t *d_partial = nullptr;      // partial sums of the planned split, reduced inside the kernel
    size_t partial_bytes = 0;
    uint32_t *d_counters = nullptr;     // one arrival counter per (tile, filter block) of the planned shape
    size_t counter_bytes = 0;
    mutable std::mutex split_mu;        // orders the launches of planned splits (the counters only grow)
    mutable uint32_t split_seq = 0;     // planned split launches enqueued so far
    int *d_status = nullptr;            // set by a kernel whose bounded wait ran out
    xgen_patconv_tuning tuning{};       // caller's overrides (xgen_patconv_plan_tuned)
    uint32_t wait_us = 2000000;         // bound of every device-side wait
    int hook_extra_arrivals = 0;        // testing aid: arrivals a planned split waits for beyond its own
    // prepared launches (shape, input address)
    mutable std::mutex cache_mu;
    mutable LaunchEntry cache[kLaunchCache];
    mutable uint64_t cache_stamp = 0;
    // device staging buffers of xgen_patconv_run_host, kept between calls (grow only)
    mutable std::mutex host_mu;
    mutable void *d_hx = nullptr, *d_hy = nullptr, *d_hb = nullptr;
    mutable size_t hx_bytes = 0, hy_bytes = 0;
    // their copies run on two streams of the handle's own, tied to the caller's stream by events
    mutable cudaStream_t s_in = nullptr, s_out = nullptr;
    mutable cudaEvent_t ev_in = nullptr, ev_run = nullptr, ev_out = nullptr;
    mutable bool host_call_before = false;
};

static void free_device_layout(xgen_patconv_packed *h) {
    if (h->d_slots) cudaFree(h->d_slots);
    if (h->d_seg_off) cudaFree(h->d_seg_off);
    if (h->d_slot_oc) cudaFree(h->d_slot_oc);
    if (h->d_status) cudaFree(h->d_status);
    h->d_slots = nullptr; h->d_seg_off = nullptr; h->d_slot_oc = nullptr; h->d_status = nullptr;
}

// Upload the host layout; the device must be current.  On the device a command slot is
// 48 bytes: {opcode, operand, -, -, w0, w0, w1, w1, w2, w2, w3, w3}; every weight twice, so
// that a 64-bit load yields the operand pair of a two-wide FMA.
static xgen_status upload_layout(xgen_patconv_packed *h) {
    const PackedHost &p = h->host;
    free_device_layout(h);
    const size_t n_slots = p.slots.size() / kSlotWords;
    std::vector<uint32_t> dev((n_slots + 2) * kDevSlotWords, 0u);    // two spare slots: look-ahead room
    for (size_t i = 0; i < n_slots; ++i) {
        const uint32_t *src = &p.slots[i * kSlotWords];
        uint32_t *dst = &dev[i * kDevSlotWords];
        dst[0] = src[0]; dst[1] = src[1];
        for (int k = 0; k < 4; ++k) dst[4 + 2 * k] = dst[5 + 2 * k] = src[4 + k];
    }
    const size_t sb = dev.size() * 4, gb = p.seg_off.size() * 4, ob = p.slot_oc.size() * 4;
    cudaError_t e = cudaMalloc(&h->d_slots, sb);
    if (e == cudaSuccess) e = cudaMalloc(&h->d_seg_off, gb);
    if (e == cudaSuccess) e = cudaMalloc(&h->d_slot_oc, ob);
    if (e == cudaSuccess) e = cudaMalloc(&h->d_status, sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(h->d_status, 0, sizeof(int));
    if (e == cudaSuccess) e = cudaMemcpy(h->d_slots, dev.data(), sb, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(h->d_seg_off, p.seg_off.data(), gb, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(h->d_slot_oc, p.slot_oc.data(), ob, cudaMemcpyHostToDevice);
    if (e != cudaSuccess) {
        xgen_status r = (e == cudaErrorMemoryAllocation) ? XGEN_ERR_ALLOC : XGEN_ERR_CUDA;
        cudaGetLastError();
        free_device_layout(h);
        return r;
    }
    return XGEN_OK;
}

// With XGEN_PATCONV_LOG set, failed CUDA calls are named on stderr.
static cudaError_t log_cuda(cudaError_t e, const char *what) {
    if (e != cudaSuccess && log_enabled())
        fprintf(stderr, "libpatconv: %s: %s\n", what, cudaGetErrorString(e));
    return e;
}

// cuTensorMapEncodeTiled, fetched through the runtime so the library does not link libcuda.
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)ptr;
        else
            cudaGetLastError();
    });
    return fn;
}

template <int DT, int STRIDE, bool FUSED, int BH>
static const void *kernel_np(int np) {
    switch (np) {
        case 4: return (const void *)patconv_kernel<DT, STRIDE, 4, FUSED, BH>;
        case 8: return (const void *)patconv_kernel<DT, STRIDE, 8, FUSED, BH>;
        case 12: return (const void *)patconv_kernel<DT, STRIDE, 12, FUSED, BH>;
        default: return (const void *)patconv_kernel<DT, STRIDE, 126, FUSED, BH>;
    }
}

template <int DT>
static const void *kernel_of(const PackedHost &p, bool fused) {
    if (p.stride == 2) return fused ? kernel_np<DT, 2, true, 4>(p.np) : kernel_np<DT, 2, false, 4>(p.np);
    if (p.bh == 2) return kernel_np<DT, 1, false, 2>(p.np);          // the small block has no fused instances
    return fused ? kernel_np<DT, 1, true, 4>(p.np) : kernel_np<DT, 1, false, 4>(p.np);
}

// The kernel instance of a packed layer, without or with the fused operators.
static const void *kernel_for(const PackedHost &p, bool fused = false) {
    if (p.dtype == XGEN_F32) return kernel_of<XGEN_F32>(p, fused);
    if (p.dtype == XGEN_F16_F32ACC) return kernel_of<XGEN_F16_F32ACC>(p, fused);
    return kernel_of<XGEN_I8_I32>(p, fused);
}

// The opt-in to large dynamic shared memory is per function and per device: do it once.
static cudaError_t allow_large_smem(const void *kern) {
    static std::mutex mu;
    static std::vector<std::pair<const void *, int>> done;
    std::lock_guard<std::mutex> lock(mu);
    int dev = 0;
    cudaGetDevice(&dev);
    const std::pair<const void *, int> key(kern, dev);
    for (const auto &k : done) if (k == key) return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemMaxDynamic);
    if (e != cudaSuccess) return log_cuda(e, "cudaFuncSetAttribute");
    done.push_back(key);
    return cudaSuccess;
}

static int next_pow2(int v) { int p = 32; while (p < v) p <<= 1; return p; }

static xgen_status layout_for(const PackedHost &p, const Geometry &g_in, int n, int hh, int ww, bool y_aligned32,
                              bool tma_ok, Layout &L) {
    const int ho = (hh + 2 - 3) / p.stride + 1, wo = (ww + 2 - 3) / p.stride + 1;
    Geometry g = g_in;
    if (g.rows) {
        // Every slot is the destination of a tensor copy of its own and must start on a
        // 128-byte boundary of shared memory: widen the staged rows (the extra columns are
        // copied, or zero-filled beyond the image, and never used) until a slot is a
        // multiple of 128 bytes.
        const int xb0 = p.dtype == XGEN_F32 ? 4 : (p.dtype == XGEN_F16_F32ACC ? 2 : 1);
        const int rc0 = p.cc * xb0 >= 16 ? p.cc : 16 / xb0;
        while ((g.tin_w * g.tin_h * rc0 * xb0) % 128 != 0) ++g.tin_w;
    }
    L.g = g;
    KParams kp{};
    kp.n = n; kp.h = hh; kp.w = ww; kp.ho = ho; kp.wo = wo; kp.c_in = p.c_in; kp.c_out = p.c_out;
    kp.J = p.J; kp.wpc = p.wpc; kp.cc = p.cc; kp.n_chunks = p.n_chunks;
    kp.lx_log = g.lx_log; kp.ly_log = g.ly_log; kp.ln_log = g.ln_log;
    kp.rows = g.rows; kp.bxn = g.bxn; kp.byn = g.byn; kp.blocks_total = g.blocks_total; kp.n_slots = g.n_slots;
    kp.tiles_x = g.tiles_x; kp.tiles_y = g.tiles_y;
    kp.tin_w = g.tin_w; kp.tin_h = g.tin_h;
    kp.pitch = g.pitch; kp.img_stride = g.img_stride; kp.plane_stride = g.plane_stride;
    kp.half_stride = g.half_stride;
    const int xb = p.dtype == XGEN_F32 ? 4 : (p.dtype == XGEN_F16_F32ACC ? 2 : 1);
    const int npix_box = g.tin_w * g.tin_h * g.n_slots;
    // A box carries at least 16 bytes of channels per pixel; a chunk may be a part of it.
    // The copy engine needs 16-byte multiples in every global stride.
    kp.rc = p.cc * xb >= 16 ? p.cc : 16 / xb;
    kp.spb = kp.rc / p.cc;
    auto magic = [](int d) { return d <= 1 ? 0u : (uint32_t)((1ull << 32) / (uint64_t)d + 1ull); };
    kp.mg_tiles_x = magic(g.tiles_x); kp.mg_tiles_y = magic(g.tiles_y);
    kp.mg_tin_w = magic(g.tin_w); kp.mg_tin_h = magic(g.tin_h); kp.mg_spb = magic(kp.spb);
    kp.mg_bxn = magic(g.bxn); kp.mg_byn = magic(g.byn);
    kp.use_tma = tma_ok && ((p.cc * xb) % 4 == 0) && (((size_t)p.c_in * xb) % 16 == 0) && g.tin_w <= 256 && g.tin_h <= 256;
    kp.box_bytes = npix_box * kp.rc * xb;
    kp.slot_bytes = g.tin_w * g.tin_h * kp.rc * xb;
    // widest aligned store per 8-channel piece: 8 words (32-byte aligned rows), 4, or scalar
    kp.vec_out = ((p.c_out % 8) == 0 && y_aligned32) ? 8 : ((p.c_out % 4) == 0 ? 4 : 0);
    const bool is_i8 = p.dtype == XGEN_I8_I32;
    const int T = p.tpix;
    kp.flush_chunks = 16777216 / (p.cc * 4 * 32640);
    if (kp.flush_chunks < 1) return XGEN_ERR_UNSUPPORTED;
    kp.fold = (is_i8 && p.int_totals) ? 1 : 0;
    kp.cols_per_warp = p.J * T * (kp.fold ? 2 : 1);
    kp.tmem_cols = next_pow2(((p.wpc + 3) / 4) * kp.cols_per_warp);
    if (kp.tmem_cols > 512) return XGEN_ERR_UNSUPPORTED;
    // Shared-memory layout (words): raw boxes | plane stages | command stages | tables | barriers.
    kp.cmd_stage_words = ((p.max_seg_slots + 2) * kDevSlotWords + 31) & ~31;
    kp.plane_stage_words = (p.cc * g.plane_stride + 31) & ~31;
    const int max_ctas = 512 / kp.tmem_cols;          // blocks per SM that tensor memory has columns for
    const size_t seg_words = ((size_t)p.n_chunks * (p.wpc + 1) + 1) & ~(size_t)1;
    auto smem_words = [&](int stages, int tma) {
        size_t w = (size_t)(tma ? kRawStages * ((kp.box_bytes / 4 + 31) & ~31) : 0);
        w += (size_t)stages * (kp.plane_stage_words + kp.cmd_stage_words);
        w += 2 * (size_t)npix_box + (tma ? 0 : ((size_t)npix_box + 1) & ~(size_t)1) + 40 * (size_t)T + seg_words;   // tables: staged pixels, output pixels (+ pooled), segments
        return w + 2 * (3 * kMaxStages + 2 * kRawStages + 2);     // + mbarriers
    };
    auto occupancy = [&](size_t words) {
        int o = (int)((size_t)kSmemPerSM / (words * 4 + 2112));     // + static and per-block reserved shared memory
        return o < max_ctas ? o : max_ctas;
    };
    if (kp.use_tma && smem_words(2, 1) * 4 > (size_t)kSmemMaxDynamic) kp.use_tma = 0;   // the raw boxes do not fit
    // Stage count: as many as fit (up to 4) without lowering the number of blocks per SM.
    int n_stages = 2;
    for (int st = 3; st <= kMaxStages; ++st)
        if (smem_words(st, kp.use_tma) * 4 <= (size_t)kSmemMaxDynamic &&
            occupancy(smem_words(st, kp.use_tma)) >= occupancy(smem_words(2, kp.use_tma))) n_stages = st;
    kp.n_stages = n_stages;
    kp.raw_stage_words = kp.use_tma ? ((kp.box_bytes / 4 + 31) & ~31) : 0;
    kp.raw_off_words = 0;
    kp.plane_off_words = kp.use_tma ? kRawStages * kp.raw_stage_words : 0;
    kp.cmd_off_words = kp.plane_off_words + n_stages * kp.plane_stage_words;
    kp.tab_off_words = kp.cmd_off_words + n_stages * kp.cmd_stage_words;
    kp.src_off_words = kp.tab_off_words + 2 * npix_box;
    kp.ptab_off_words = kp.src_off_words + (kp.use_tma ? 0 : ((npix_box + 1) & ~1));
    kp.seg_off_words = kp.ptab_off_words + 40 * T;
    kp.mbar_off_words = kp.seg_off_words + (int)seg_words;
    size_t smem = smem_words(n_stages, kp.use_tma) * 4;
    // Never let more blocks share an SM than tensor memory has columns for.
    const size_t floor_bytes = (size_t)kSmemPerSM / (max_ctas + 1);
    if (smem < floor_bytes) smem = floor_bytes;
    if (smem > (size_t)kSmemMaxDynamic) return XGEN_ERR_UNSUPPORTED;
    kp.out_elems = (size_t)n * ho * wo * p.c_out;
    L.kp = kp;
    L.smem = smem;
    L.items = g.tiles * p.n_blocks;
    return XGEN_OK;
}

// The launch layout of a shape.  Row tiling is taken where it covers clearly more of the pixel
// slots than the best grid tiling (it stages more halo per pixel, so a small gain does not pay)
// and where its larger staged tile still fits shared memory together with the copy engine's
// boxes; otherwise grid tiling.  *rows_wanted tells the caller that row tiling was preferred
// (whether or not it fitted), so that a planner may try again with smaller channel chunks.
static xgen_status make_layout(const PackedHost &p, int n, int hh, int ww, bool y_aligned32, bool tma_ok, Layout &L,
                               bool *rows_wanted = nullptr) {
    const int ho = (hh + 2 - 3) / p.stride + 1, wo = (ww + 2 - 3) / p.stride + 1;
    const Geometry grid = grid_geometry(n, ho, wo, p.stride, p.bh);
    Geometry rows;
    const bool want = row_geometry(n, ho, wo, p.stride, p.bh, rows) && rows.covered > 1.08 * grid.covered;
    if (rows_wanted) *rows_wanted = want;
    const xgen_status gs = layout_for(p, grid, n, hh, ww, y_aligned32, tma_ok, L);
    if (want) {
        Layout Lr;
        if (layout_for(p, rows, n, hh, ww, y_aligned32, tma_ok, Lr) == XGEN_OK &&
            (gs != XGEN_OK || Lr.kp.use_tma >= L.kp.use_tma)) {
            L = Lr;
            return XGEN_OK;
        }
    }
    return gs;
}

// 1 KB rows of partial sums one (item, split) writes in a split run reduced inside the kernel.
static size_t rows_per_item(const PackedHost &p) {
    return (size_t)p.wpc * ((p.J + 7) / 8) * p.tpix;
}

// The prepared launch of (shape, input address, alignment class of y): from the handle's
// small cache, or built now (geometry, shared-memory layout, tensor map) and kept.
static xgen_status prepared_launch(const xgen_patconv_packed *h, const void *x, int n, int hh, int ww, bool y32,
                                   Layout &L, CUtensorMap &tm) {
    std::lock_guard<std::mutex> lock(h->cache_mu);
    LaunchEntry *victim = &h->cache[0];
    for (LaunchEntry &e : h->cache) {
        if (e.stamp && e.n == n && e.h == hh && e.w == ww && e.x == x && e.y32 == y32) {
            e.stamp = ++h->cache_stamp;
            L = e.L; tm = e.tm;
            return XGEN_OK;
        }
        if (e.stamp < victim->stamp) victim = &e;
    }
    const PackedHost &p = h->host;
    EncodeTiledFn encode = h->tuning.no_copy_engine ? nullptr : encode_tiled_fn();
    LaunchEntry ne;
    xgen_status ls = make_layout(p, n, hh, ww, y32, encode != nullptr, ne.L);
    if (ls != XGEN_OK) return ls;
    memset(&ne.tm, 0, sizeof(ne.tm));
    if (ne.L.kp.use_tma) {
        const Geometry &g = ne.L.g;
        const int xb = p.dtype == XGEN_F32 ? 4 : (p.dtype == XGEN_F16_F32ACC ? 2 : 1);
        const cuuint64_t gdim[4] = {(cuuint64_t)p.c_in, (cuuint64_t)ww, (cuuint64_t)hh, (cuuint64_t)n};
        const cuuint64_t gstr[3] = {(cuuint64_t)p.c_in * xb, (cuuint64_t)ww * p.c_in * xb, (cuuint64_t)hh * ww * p.c_in * xb};
        const cuuint32_t box[4] = {(cuuint32_t)ne.L.kp.rc, (cuuint32_t)g.tin_w, (cuuint32_t)g.tin_h, (cuuint32_t)(g.rows ? 1 : g.n_slots)};
        const cuuint32_t estr[4] = {1, 1, 1, 1};
        const CUtensorMapDataType dt = p.dtype == XGEN_F32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                                     : (p.dtype == XGEN_F16_F32ACC ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8);
        const CUresult cr = encode(&ne.tm, dt, 4, const_cast<void *>(x), gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                   CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (cr != CUDA_SUCCESS) {          // stage with plain loads instead
            if (log_enabled()) fprintf(stderr, "libpatconv: cuTensorMapEncodeTiled failed (%d)\n", (int)cr);
            memset(&ne.tm, 0, sizeof(ne.tm));
            ls = make_layout(p, n, hh, ww, y32, false, ne.L);
            if (ls != XGEN_OK) return ls;
        }
    }
    ne.n = n; ne.h = hh; ne.w = ww; ne.x = x; ne.y32 = y32;
    ne.stamp = ++h->cache_stamp;
    *victim = ne;
    L = ne.L; tm = ne.tm;
    return XGEN_OK;
}

static void forget_prepared_launches(xgen_patconv_packed *h) {
    std::lock_guard<std::mutex> lock(h->cache_mu);
    for (LaunchEntry &e : h->cache) e.stamp = 0;
}

// Where a run keeps the partial sums of a split, when the caller (not the plan) decides.
struct SplitChoice { int splits, chunks_per_split; uint32_t *partial; };

static xgen_status run_layer(const xgen_patconv_packed *h, const void *x, int32_t n, int32_t hh, int32_t ww,
                             const void *bias, int32_t relu, void *y, void *stream, const SplitChoice *forced,
                             const xgen_patconv_epilogue *ep = nullptr) {
    if (!h || !x || !y) return XGEN_ERR_INVALID_ARG;
    if (((uintptr_t)x & 15) || ((uintptr_t)y & 15) || ((uintptr_t)bias & 3)) return XGEN_ERR_INVALID_ARG;
    if (n < 1 || hh < 1 || ww < 1) return XGEN_ERR_SHAPE;
    const PackedHost &p = h->host;
    if (h->device < 0) return XGEN_ERR_CUDA;
    const int ho = (hh + 2 - 3) / p.stride + 1, wo = (ww + 2 - 3) / p.stride + 1;
    if ((int64_t)n * hh * ww * p.c_in > 0x7FFFFFFFLL || (int64_t)n * ho * wo * p.c_out > 0x7FFFFFFFLL) return XGEN_ERR_SHAPE;
    const int xb = p.dtype == XGEN_F32 ? 4 : (p.dtype == XGEN_F16_F32ACC ? 2 : 1);
    // operators fused behind the convolution
    const int pool = ep ? ep->pool : 0;
    const void *residual = ep ? ep->residual_dev : nullptr;
    const float *rq_scale = ep ? ep->requant_scale_dev : nullptr;
    if (ep) {
        if (forced || p.bh != 4) return XGEN_ERR_UNSUPPORTED;
        if (pool != 0 && pool != 2) return XGEN_ERR_UNSUPPORTED;
        if (pool == 2 && ((ho & 1) || (wo & 1))) return XGEN_ERR_SHAPE;
        if (rq_scale && p.dtype != XGEN_I8_I32) return XGEN_ERR_UNSUPPORTED;
        if (((uintptr_t)residual & 15) || ((uintptr_t)rq_scale & 3)) return XGEN_ERR_INVALID_ARG;
        relu = ep->relu;
    }
    const int po = pool == 2 ? ho / 2 : ho, pw = pool == 2 ? wo / 2 : wo;
    {
        const char *xa = (const char *)x, *ya = (const char *)y, *ra = (const char *)residual;
        const int yb = rq_scale ? 1 : (p.dtype == XGEN_F16_F32ACC ? 2 : 4), rb = p.dtype == XGEN_F16_F32ACC ? 2 : 4;
        const char *xe = xa + (size_t)n * hh * ww * p.c_in * xb, *ye = ya + (size_t)n * po * pw * p.c_out * yb;
        if (xa < ye && ya < xe) return XGEN_ERR_INVALID_ARG;   // overlap
        if (ra) {
            const char *re = ra + (size_t)n * ho * wo * p.c_out * rb;
            if (ra < ye && ya < re) return XGEN_ERR_INVALID_ARG;
        }
    }
    Layout L;
    CUtensorMap tm;
    xgen_status ls = prepared_launch(h, x, n, hh, ww, ((uintptr_t)y & 31) == 0, L, tm);
    if (ls != XGEN_OK) return ls;
    KParams kp = L.kp;
    const size_t smem = L.smem;
    kp.x = x; kp.y = y; kp.bias = bias;
    kp.slots = h->d_slots; kp.seg_off = h->d_seg_off; kp.slot_oc = h->d_slot_oc;
    kp.relu = relu ? 1 : 0;
    kp.residual = residual; kp.rq_scale = rq_scale; kp.rq_zero = ep ? ep->requant_zero_point : 0;
    kp.pool = pool; kp.po = po; kp.pw = pw;
    kp.status = h->d_status;
    kp.wait_us = h->wait_us;
    // Split runs: a caller-chosen split keeps [split][output] sums for a second kernel; the
    // planned split is reduced inside the kernel (rows of partial sums plus arrival counters).
    const bool planned = !forced && h->plan_splits > 1 && h->plan_n == n && h->plan_h == hh && h->plan_w == ww &&
                         h->d_partial && h->d_counters;
    const bool split = forced ? forced->splits > 1 : planned;
    const int n_splits = split ? (forced ? forced->splits : h->plan_splits) : 1;
    // block numbering: whole items first, then the split items, n_splits blocks each
    const int whole = split ? (forced ? 0 : h->plan_whole) : L.items;
    const int64_t n_blocks_launch = (int64_t)whole + (int64_t)(L.items - whole) * n_splits;
    if (n_blocks_launch > 0x7FFFFFFFLL) return XGEN_ERR_SHAPE;
    auto magic = [](int d) { return d <= 1 ? 0u : (uint32_t)((1ull << 32) / (uint64_t)d + 1ull); };
    kp.whole_items = whole;
    kp.n_splits = n_splits;
    kp.mg_splits = magic(n_splits);
    kp.n_tiles = L.g.tiles;
    kp.mg_tiles = magic(L.g.tiles);
    kp.chunks_per_split = split ? (forced ? forced->chunks_per_split : h->plan_cps) : p.n_chunks;
    kp.partial = (split && forced) ? forced->partial : nullptr;

    int prev = 0;
    if (cudaGetDevice(&prev) != cudaSuccess) return XGEN_ERR_CUDA;
    if (prev != h->device && cudaSetDevice(h->device) != cudaSuccess) return XGEN_ERR_CUDA;
    dim3 grid((unsigned)n_blocks_launch, 1, 1), block((unsigned)((p.wpc + kProducerWarps) * 32), 1, 1);
    cudaStream_t st = (cudaStream_t)stream;
    if (log_enabled())
        fprintf(stderr, "libpatconv: %u blocks = %d whole items + %d items x %d splits (%d tiles x %d filter blocks), %u threads, %zu bytes shared, %d stages, %s lanes %dx%dx%d, tile in %dx%d x %d slots, tma %d, cc %d, fused split %d\n",
                grid.x, whole, L.items - whole, n_splits, L.g.tiles, p.n_blocks, block.x, smem, kp.n_stages, L.g.rows ? "row tiling," : "grid tiling,",
                L.g.rows ? L.g.bxn : 1 << L.g.lx_log, L.g.rows ? 1 : 1 << L.g.ly_log, L.g.rows ? 1 : 1 << L.g.ln_log,
                L.g.tin_w, L.g.tin_h, L.g.n_slots, kp.use_tma, p.cc, planned ? 1 : 0);
    const void *kern = kernel_for(p, ep != nullptr);
    cudaError_t e = allow_large_smem(kern);
    if (e == cudaSuccess) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
        // Programmatic stream serialisation: this kernel may be scheduled while its predecessor
        // in the stream drains (it waits for it, griddepcontrol.wait, before touching memory), and
        // it lets its successor do the same.  A dependent grid starts only after every block of
        // this one has started, so the blocks of a split, which wait for each other and which the
        // planner keeps within what the GPU holds at once, are never kept out by a successor.
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = h->tuning.no_launch_overlap ? 0 : 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        void *args[2] = {(void *)&kp, (void *)&tm};
        if (planned) {
            // The arrival counters of a planned split only grow: launch k waits for k x splits
            // arrivals.  The sequence number moves on only when the launch was accepted.
            std::lock_guard<std::mutex> lock(h->split_mu);
            kp.ws = h->d_partial;
            kp.counters = h->d_counters;
            kp.last_reduces = h->plan_last ? 1 : 0;
            kp.target = (h->split_seq + 1u) * (uint32_t)n_splits + (h->plan_last ? 0u : (uint32_t)h->hook_extra_arrivals);
            e = cudaLaunchKernelExC(&cfg, kern, args);
            if (e == cudaSuccess) e = cudaGetLastError();
            if (e == cudaSuccess) ++h->split_seq;
        } else {
            e = cudaLaunchKernelExC(&cfg, kern, args);
            if (e == cudaSuccess) e = cudaGetLastError();
        }
        e = log_cuda(e, "kernel launch");
    }
    if (e == cudaSuccess && split && forced) {
        const int vec = kp.vec_out >= 4 ? 1 : 0;
        const size_t items = vec ? kp.out_elems / 4 : kp.out_elems;
        const unsigned blocks = (unsigned)((items + 255) / 256);
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(blocks, 1, 1); cfg.blockDim = dim3(256, 1, 1); cfg.dynamicSmemBytes = 0; cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        const uint32_t *part_c = forced->partial;
        const size_t oe = kp.out_elems;
        const int co = p.c_out, rl = kp.relu;
        const void *bias_c = bias;
        if (p.dtype == XGEN_F32)
            e = cudaLaunchKernelEx(&cfg, patconv_reduce_kernel<XGEN_F32>, part_c, n_splits, oe, co, bias_c, rl, y, vec);
        else if (p.dtype == XGEN_F16_F32ACC)
            e = cudaLaunchKernelEx(&cfg, patconv_reduce_kernel<XGEN_F16_F32ACC>, part_c, n_splits, oe, co, bias_c, rl, y, vec);
        else
            e = cudaLaunchKernelEx(&cfg, patconv_reduce_kernel<XGEN_I8_I32>, part_c, n_splits, oe, co, bias_c, rl, y, vec);
        if (e == cudaSuccess) e = cudaGetLastError();
        e = log_cuda(e, "reduce launch");
        if (e == cudaSuccess) g_launches.fetch_add(1);
    }
    if (prev != h->device) cudaSetDevice(prev);
    if (e != cudaSuccess) return XGEN_ERR_CUDA;
    g_launches.fetch_add(1);
    return XGEN_OK;
}

// The library's own scratch for xgen_patconv_run_static_scratch: partial sums of a split run.
// It lives in every CUDA context that loads this library, until the process exits.
static __device__ __align__(256) uint32_t g_static_scratch[XGEN_PATCONV_STATIC_SCRATCH_BYTES / 4];
static uint32_t *g_static_scratch_addr[64];        // device address per device ordinal, resolved once
static std::mutex g_static_scratch_mutex;

extern "C" {

const char *xgen_strerror(xgen_status s) {
    switch (s) {
        case XGEN_OK: return "ok";
        case XGEN_ERR_INVALID_ARG: return "invalid argument";
        case XGEN_ERR_BAD_PATTERN: return "bad pattern mask or pattern id";
        case XGEN_ERR_SHAPE: return "shape out of range";
        case XGEN_ERR_UNSUPPORTED: return "unsupported configuration";
        case XGEN_ERR_ALLOC: return "allocation failed";
        case XGEN_ERR_CUDA: return "CUDA error";
        case XGEN_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

int64_t xgen_patconv_launch_count(void) { return g_launches.load(); }

xgen_status xgen_patconv_pack(const xgen_patconv_desc *desc, const void *dense_w_host,
                              const int16_t *pattern_id_host, int device, xgen_patconv_packed **out) {
    if (!desc || !out) return XGEN_ERR_INVALID_ARG;
    *out = nullptr;
    xgen_patconv_packed *h = new (std::nothrow) xgen_patconv_packed();
    if (!h) return XGEN_ERR_ALLOC;
    xgen_status st;
    try {
        st = parse_layer(*desc, dense_w_host, pattern_id_host, h->host);
        PackConfig cfg{};
        if (st == XGEN_OK) {
            cfg = choose_pack_config(desc->c_in, desc->c_out, desc->dtype, desc->stride, h->host.int_totals);
            if (desc->dtype == XGEN_I8_I32 && cfg.channels_per_chunk < 4) cfg.channels_per_chunk = 4;
            st = build_layout(h->host, cfg);
        }
        // A stage of the kernel's pipeline holds the commands of one chunk for the whole
        // block: halve the chunk until the longest segment fits the command buffer.
        while (st == XGEN_OK && cfg.channels_per_chunk > 4 &&
               (size_t)h->host.max_seg_slots * kDevSlotBytes > kCmdStageBudget) {
            cfg.channels_per_chunk /= 2;
            st = build_layout(h->host, cfg);
        }
    } catch (const std::bad_alloc &) {
        st = XGEN_ERR_ALLOC;
    }
    if (st != XGEN_OK) { delete h; return st; }
    if (device >= 0) {
        int prev = 0;
        if (cudaGetDevice(&prev) != cudaSuccess || cudaSetDevice(device) != cudaSuccess) { delete h; return XGEN_ERR_CUDA; }
        xgen_status us = upload_layout(h);
        cudaSetDevice(prev);
        if (us != XGEN_OK) { delete h; return us; }
        h->device = device;
    }
    *out = h;
    return XGEN_OK;
}

void xgen_patconv_free(xgen_patconv_packed *h) {
    if (!h) return;
    free_device_layout(h);
    if (h->d_partial) cudaFree(h->d_partial);
    if (h->d_counters) cudaFree(h->d_counters);
    if (h->d_hx) cudaFree(h->d_hx);
    if (h->d_hy) cudaFree(h->d_hy);
    if (h->d_hb) cudaFree(h->d_hb);
    if (h->s_in) cudaStreamDestroy(h->s_in);
    if (h->s_out) cudaStreamDestroy(h->s_out);
    if (h->ev_in) cudaEventDestroy(h->ev_in);
    if (h->ev_run) cudaEventDestroy(h->ev_run);
    if (h->ev_out) cudaEventDestroy(h->ev_out);
    delete h;
}

xgen_status xgen_patconv_out_shape(const xgen_patconv_packed *h, int32_t hh, int32_t ww, int32_t *ho, int32_t *wo) {
    if (!h || !ho || !wo) return XGEN_ERR_INVALID_ARG;
    if (hh < 1 || ww < 1) return XGEN_ERR_SHAPE;
    *ho = (hh + 2 - 3) / h->host.stride + 1;
    *wo = (ww + 2 - 3) / h->host.stride + 1;
    return XGEN_OK;
}

xgen_status xgen_patconv_query(const xgen_patconv_packed *h, xgen_patconv_stats *s) {
    if (!h || !s) return XGEN_ERR_INVALID_ARG;
    *s = h->host.stats;
    return XGEN_OK;
}

xgen_status xgen_patconv_view(const xgen_patconv_packed *h, xgen_patconv_host_view *v) {
    if (!h || !v) return XGEN_ERR_INVALID_ARG;
    v->slots = h->host.slots.data();
    v->n_slots = (int64_t)(h->host.slots.size() / kSlotWords);
    v->seg_off = h->host.seg_off.data();
    v->slot_oc = h->host.slot_oc.data();
    v->compiled_masks = h->host.masks.data();
    return XGEN_OK;
}

xgen_status xgen_patconv_last_status(const xgen_patconv_packed *h, void *stream) {
    if (!h) return XGEN_ERR_INVALID_ARG;
    cudaError_t e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) return XGEN_ERR_CUDA;
    if (h->s_out && cudaStreamSynchronize(h->s_out) != cudaSuccess) return XGEN_ERR_CUDA;   // copies out of host-buffer calls
    if (cudaGetLastError() != cudaSuccess) return XGEN_ERR_CUDA;
    if (h->d_status) {
        // a kernel whose bounded wait ran out leaves a mark here
        int flag = 0;
        if (cudaMemcpy(&flag, h->d_status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return XGEN_ERR_CUDA;
        if (flag) {
            cudaMemset(h->d_status, 0, sizeof(int));
            // a run that gave up may have left the arrival counters of a split half way
            std::lock_guard<std::mutex> lock(h->split_mu);
            if (h->d_counters) cudaMemset(h->d_counters, 0, h->counter_bytes);
            h->split_seq = 0;
            return XGEN_ERR_TIMEOUT;
        }
    }
    return XGEN_OK;
}

// What a launch of this shape looks like with the handle as it stands.
xgen_status xgen_patconv_plan_info(const xgen_patconv_packed *h, int32_t n, int32_t hh, int32_t ww,
                                   xgen_patconv_plan_stats *out) {
    if (!h || !out) return XGEN_ERR_INVALID_ARG;
    if (n < 1 || hh < 1 || ww < 1) return XGEN_ERR_SHAPE;
    const PackedHost &p = h->host;
    Layout L;
    const bool tma_ok = !h->tuning.no_copy_engine && (h->device < 0 || encode_tiled_fn() != nullptr);
    xgen_status ls = make_layout(p, n, hh, ww, true, tma_ok, L);
    if (ls != XGEN_OK) return ls;
    const bool planned = h->plan_splits > 1 && h->plan_n == n && h->plan_h == hh && h->plan_w == ww;
    memset(out, 0, sizeof(*out));
    out->splits = planned ? h->plan_splits : 1;
    out->chunks_per_split = planned ? h->plan_cps : p.n_chunks;
    out->tiles = L.g.tiles;
    out->filter_blocks = p.n_blocks;
    out->items = L.items;
    out->whole_items = planned ? h->plan_whole : L.items;
    out->blocks = out->whole_items + (L.items - out->whole_items) * out->splits;
    out->threads_per_block = (p.wpc + kProducerWarps) * 32;
    out->row_tiling = L.g.rows;
    out->lanes_x = L.g.rows ? L.g.bxn : 1 << L.g.lx_log; out->lanes_y = L.g.rows ? 1 : 1 << L.g.ly_log;
    out->lanes_n = L.g.rows ? 1 : 1 << L.g.ln_log;
    out->covered = L.g.covered;
    out->pixels_per_lane = p.tpix;
    out->stages = L.kp.n_stages;
    out->uses_copy_engine = L.kp.use_tma;
    out->shared_bytes = (int64_t)L.smem;
    out->last_arriver = planned && h->plan_last ? 1 : 0;
    out->reserved = 0;
    out->workspace_bytes = planned ? (int64_t)((size_t)(L.items - h->plan_whole) * (size_t)h->plan_splits * rows_per_item(p) * 1024) : 0;
    return XGEN_OK;
}

xgen_status xgen_patconv_plan_tuned(xgen_patconv_packed *h, int32_t n, int32_t hh, int32_t ww,
                                    const xgen_patconv_tuning *tuning) {
    if (!h) return XGEN_ERR_INVALID_ARG;
    if (n < 1 || hh < 1 || ww < 1) return XGEN_ERR_SHAPE;
    if (h->device < 0) return XGEN_ERR_CUDA;
    if (tuning && (tuning->splits < 0 || tuning->wait_limit_ms < 0 || tuning->reduce_mode < 0 || tuning->reduce_mode > 2 ||
                   (tuning->channels_per_chunk != 0 && tuning->channels_per_chunk != 4 && tuning->channels_per_chunk != 8 &&
                    tuning->channels_per_chunk != 16) ||
                   tuning->groups_per_block < 0 || tuning->groups_per_block > (int)kMaxWarps))
        return XGEN_ERR_INVALID_ARG;
    const PackedHost &p = h->host;
    const int ho = (hh + 2 - 3) / p.stride + 1, wo = (ww + 2 - 3) / p.stride + 1;
    if ((int64_t)n * ho * wo * p.c_out > 0x7FFFFFFFLL) return XGEN_ERR_SHAPE;
    const xgen_patconv_tuning tn = tuning ? *tuning : xgen_patconv_tuning{};
    const bool tma_ok = !tn.no_copy_engine && encode_tiled_fn() != nullptr;
    int prev = 0;
    if (cudaGetDevice(&prev) != cudaSuccess || cudaSetDevice(h->device) != cudaSuccess) return XGEN_ERR_CUDA;
    xgen_status rs = XGEN_OK;
    // Rebuild the command stream for another grouping (the kept weights are still in the handle)
    // and upload it again; every later run of the handle uses the new layout.
    auto relayout = [&](PackConfig cfg) {
        xgen_status st = cudaDeviceSynchronize() == cudaSuccess ? XGEN_OK : XGEN_ERR_CUDA;
        try {
            if (st == XGEN_OK) st = build_layout(h->host, cfg);
            while (st == XGEN_OK && cfg.channels_per_chunk > 4 &&
                   (size_t)h->host.max_seg_slots * kDevSlotBytes > kCmdStageBudget) {
                cfg.channels_per_chunk /= 2;
                st = build_layout(h->host, cfg);
            }
        } catch (const std::bad_alloc &) {
            st = XGEN_ERR_ALLOC;
        }
        if (st == XGEN_OK) st = upload_layout(h);
        forget_prepared_launches(h);
        return st;
    };
    // Grouping of the command stream for this shape.  A stride-1 thread owns 4x4 output pixels; a
    // shape that leaves most lanes of every such tiling idle (a single 14x14 image fills 38 % of a
    // warp's 512 pixel slots) runs with 4x2 pixels per thread and 16 filters per warp instead, if
    // that at least covers 1.4 times as much.  Integer layers with int32 totals keep the large
    // block (their second tensor-memory row leaves no room for 16 filters).  The caller's tuning
    // may name the channels per chunk and the filter groups per block.
    {
        auto covered = [&](int bh) {
            const Geometry g = grid_geometry(n, ho, wo, p.stride, bh);
            Geometry r;
            return row_geometry(n, ho, wo, p.stride, bh, r) ? std::max(g.covered, r.covered) : g.covered;
        };
        const bool small = p.stride == 1 && !p.int_totals && !tn.no_small_blocks && covered(4) < 0.55 && covered(2) >= 1.4 * covered(4);
        PackConfig cfg = choose_pack_config(p.c_in, p.c_out, p.dtype, p.stride, p.int_totals);
        if (p.dtype == XGEN_I8_I32 && cfg.channels_per_chunk < 4) cfg.channels_per_chunk = 4;
        if (small) {
            cfg.block_rows = 2;
            cfg.filters_per_group = 16;
            // eight groups per block: twice the blocks of output channels and half the channel
            // splits of sixteen (measured 7 % faster on 512 -> 512 at 14x14)
            cfg.groups_per_block = std::min((p.c_out + 15) / 16, 8);
        }
        if (tn.channels_per_chunk) cfg.channels_per_chunk = tn.channels_per_chunk;
        if (tn.groups_per_block) cfg.groups_per_block = std::min(tn.groups_per_block, cfg.groups_per_block);
        const bool asked = tn.channels_per_chunk || tn.groups_per_block || h->layout_asked;
        const bool differs = cfg.filters_per_group != p.J || cfg.groups_per_block != p.wpc || cfg.block_rows != p.bh ||
                             (asked && cfg.channels_per_chunk != p.cc);
        if (small != (p.bh == 2) || (asked && differs)) {
            rs = relayout(cfg);
            h->layout_asked = tn.channels_per_chunk || tn.groups_per_block;
            if (rs != XGEN_OK) { cudaSetDevice(prev); h->plan_splits = 1; h->plan_n = 0; return rs; }
        }
    }
    Layout L;
    bool rows_wanted = false;
    xgen_status ls = make_layout(p, n, hh, ww, true, tma_ok, L, &rows_wanted);
    if (ls != XGEN_OK) { cudaSetDevice(prev); return ls; }
    if (rows_wanted && !L.g.rows && p.cc > 4 && !tn.channels_per_chunk) {
        // Row tiling covers more of this shape but its staged tile (one slot per block row)
        // does not fit with the chunk size chosen at pack time: half the channels per chunk.
        PackConfig cfg{p.J, p.wpc, p.cc / 2};
        cfg.block_rows = p.bh;
        rs = relayout(cfg);
        if (rs == XGEN_OK) rs = make_layout(p, n, hh, ww, true, tma_ok, L);
        if (rs != XGEN_OK) { cudaSetDevice(prev); h->plan_splits = 1; h->plan_n = 0; return rs; }
    }
    int sms = 148, bps = 0;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, h->device);
    const void *kern = kernel_for(p);
    if (allow_large_smem(kern) != cudaSuccess ||
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&bps, kern, (p.wpc + kProducerWarps) * 32, L.smem) != cudaSuccess) {
        cudaGetLastError();
        rs = XGEN_ERR_CUDA;
    }
    bps = std::min(bps, 512 / L.kp.tmem_cols);
    // The splits of an item wait for each other inside the kernel, so all blocks of split items
    // must be resident at once: (split items) x splits <= SMs x blocks per SM.  Two cases.
    // Few items (not more than the GPU holds blocks): every item is split, and the split count
    // comes from a small cost model (cycles): a block costs a fixed prologue and epilogue plus
    // its multiply-adds at the rate an SM sustains with the warps it then hosts; a split adds
    // the exchange of the partial sums.  Many items: the GPU works through them in waves of
    // `capacity` blocks, and the last wave is only partly filled; the items of that last wave
    // are split (they are numbered last, so their blocks start as the wave before them drains),
    // all earlier items run whole.
    const int64_t capacity = std::max<int64_t>(1, (int64_t)sms * bps);
    const double slot_macs_item = 4.0 * (double)p.stats.kernels_surviving / (double)p.n_blocks * 32.0 * p.tpix;
    auto sm_rate = [&](int warps) { return 50.0 * std::pow((double)std::min(warps, 16) / 16.0, 0.65); };   // multiply-adds per cycle
    // Cost model, cycles.  A block costs a fixed prologue and epilogue plus its multiply-adds at the
    // rate an SM sustains with the warps it then hosts.  Waiting splits add the exchange of the
    // partial sums (every block writes its sums, waits, and reduces a share).
    auto parts_of = [&](int64_t k) { const int c = (int)((p.n_chunks + k - 1) / k); return (int64_t)((p.n_chunks + c - 1) / c); };
    auto work_of = [&](int64_t k) { return slot_macs_item * (double)((p.n_chunks + k - 1) / k) / (double)p.n_chunks; };
    const size_t ws_limit = (size_t)1 << 30;                    // no plan takes more than 1 GiB of workspace
    auto ws_bytes = [&](int64_t n_items, int64_t k) { return (size_t)n_items * (size_t)parts_of(k) * rows_per_item(p) * 1024; };
    int64_t splits = 1, whole = L.items;
    bool last = false;
    // The splits of an item that wait for each other inside the kernel must all be resident at
    // once: (split items) x splits <= SMs x blocks per SM.  Two cases.  Few items (not more than
    // the GPU holds blocks): every item is split.  Many items: the GPU works through them in waves
    // of `capacity` blocks, and the last wave is only partly filled; the items of that last wave
    // are split (they are numbered last, so their blocks start as the wave before them drains),
    // all earlier items run whole.
    const bool few = L.items <= capacity;
    const int64_t rest = few ? L.items : L.items % capacity;     // the items that may be split
    if (rest > 0) {
        const int64_t max_wait = std::max<int64_t>(1, std::min<int64_t>(p.n_chunks, capacity / rest));
        auto t_wait = [&](int64_t k) {
            const int64_t parts = parts_of(k), blocks = rest * parts;
            const int per_sm = few ? (int)((blocks + sms - 1) / sms) : bps;
            double t = 9000.0 + work_of(k) * (few ? per_sm : 1) / sm_rate(per_sm * p.wpc);
            if (parts > 1) t += 5000.0 + 150.0 * (double)parts;
            return t;
        };
        const double margin = few ? 0.97 : 0.9;                  // a split has to pay for itself
        double best_t = t_wait(1);
        // Splits added up by the last arriver are never the planner's own choice: with more blocks
        // than the GPU holds at once they run in waves, and on the shapes tried (items between a
        // half and three times the SM count, 2 to 8 splits) every such plan measured slower than
        // the best plan of whole items and waiting splits.  They are there for callers that must
        // run planned launches of several handles at the same time (reduce_mode = 2).
        for (int64_t k = 2; k <= max_wait; ++k) {
            const double t = t_wait(k);
            if (t < margin * best_t) { best_t = t; splits = k; }
        }
        last = tn.reduce_mode == 2 && splits > 1;                // the same count, nobody waiting
        if (tn.splits >= 1) {
            if (tn.reduce_mode == 2) {
                last = tn.splits > 1;
                splits = std::min<int64_t>(tn.splits, p.n_chunks);
                while (splits > 1 && ws_bytes(rest, splits) > ws_limit) --splits;
            } else {
                last = false;
                splits = std::max<int64_t>(1, std::min<int64_t>(tn.splits, max_wait));
            }
        }
        whole = splits > 1 ? L.items - rest : L.items;
    }
    const int cps = (int)((p.n_chunks + splits - 1) / splits);
    splits = (p.n_chunks + cps - 1) / cps;
    if (splits <= 1) { whole = L.items; last = false; }
    const int64_t split_items = L.items - whole;
    if (rs == XGEN_OK && cudaDeviceSynchronize() != cudaSuccess) rs = XGEN_ERR_CUDA;
    if (rs == XGEN_OK && splits > 1) {
        const size_t need = (size_t)split_items * (size_t)splits * rows_per_item(p) * 1024;
        const size_t need_c = (size_t)split_items * sizeof(uint32_t);
        if (need > h->partial_bytes) {
            if (h->d_partial) cudaFree(h->d_partial);
            h->d_partial = nullptr; h->partial_bytes = 0;
            if (cudaMalloc(&h->d_partial, need) != cudaSuccess) { cudaGetLastError(); rs = XGEN_ERR_ALLOC; }
            else h->partial_bytes = need;
        }
        if (rs == XGEN_OK && need_c > h->counter_bytes) {
            if (h->d_counters) cudaFree(h->d_counters);
            h->d_counters = nullptr; h->counter_bytes = 0;
            if (cudaMalloc(&h->d_counters, need_c) != cudaSuccess) { cudaGetLastError(); rs = XGEN_ERR_ALLOC; }
            else h->counter_bytes = need_c;
        }
        if (rs == XGEN_OK && cudaMemset(h->d_counters, 0, h->counter_bytes) != cudaSuccess) rs = XGEN_ERR_CUDA;
    }
    cudaSetDevice(prev);
    {
        std::lock_guard<std::mutex> lock(h->split_mu);
        h->split_seq = 0;
    }
    forget_prepared_launches(h);
    if (rs != XGEN_OK) { h->plan_splits = 1; h->plan_n = 0; return rs; }
    h->tuning = tn;
    h->wait_us = tn.wait_limit_ms > 0 ? (uint32_t)std::min<int64_t>((int64_t)tn.wait_limit_ms * 1000, 60000000) : 2000000u;
    h->plan_n = n; h->plan_h = hh; h->plan_w = ww;
    h->plan_splits = (int)splits; h->plan_cps = cps; h->plan_whole = (int)whole; h->plan_last = last;
    return XGEN_OK;
}

xgen_status xgen_patconv_plan(xgen_patconv_packed *h, int32_t n, int32_t hh, int32_t ww) {
    return xgen_patconv_plan_tuned(h, n, hh, ww, nullptr);
}

xgen_status xgen_patconv_test_expect_arrivals(xgen_patconv_packed *h, int32_t extra) {
    if (!h || extra < 0) return XGEN_ERR_INVALID_ARG;
    h->hook_extra_arrivals = extra;
    return XGEN_OK;
}

xgen_status xgen_patconv_run(const xgen_patconv_packed *h, const void *x, int32_t n, int32_t hh, int32_t ww,
                             const void *bias, int32_t relu, void *y, void *stream) {
    return run_layer(h, x, n, hh, ww, bias, relu, y, stream, nullptr);
}

xgen_status xgen_patconv_run_fused(const xgen_patconv_packed *h, const void *x, int32_t n, int32_t hh, int32_t ww,
                                   const void *bias, const xgen_patconv_epilogue *ep, void *y, void *stream) {
    if (!ep) return XGEN_ERR_INVALID_ARG;
    return run_layer(h, x, n, hh, ww, bias, ep->relu, y, stream, nullptr, ep);
}

xgen_status xgen_patconv_run_static_scratch(const xgen_patconv_packed *h, const void *x, int32_t n, int32_t hh,
                                            int32_t ww, const void *bias, int32_t relu, void *y,
                                            int32_t splits, void *stream) {
    if (!h || !x || !y || splits < 1) return XGEN_ERR_INVALID_ARG;
    if (n < 1 || hh < 1 || ww < 1) return XGEN_ERR_SHAPE;
    if (h->device < 0 || h->device >= 64) return XGEN_ERR_CUDA;
    const PackedHost &p = h->host;
    const int ho = (hh + 2 - 3) / p.stride + 1, wo = (ww + 2 - 3) / p.stride + 1;
    const int64_t out_elems = (int64_t)n * ho * wo * p.c_out;
    if (out_elems > 0x7FFFFFFFLL) return XGEN_ERR_SHAPE;
    if (splits > p.n_chunks) splits = p.n_chunks;
    const int cps = (p.n_chunks + splits - 1) / splits;
    const int eff = (p.n_chunks + cps - 1) / cps;                 // splits that actually get chunks
    if (eff > 1 && (uint64_t)out_elems * 4u * (uint64_t)eff > (uint64_t)XGEN_PATCONV_STATIC_SCRATCH_BYTES) {
        if (log_enabled())
            fprintf(stderr, "libpatconv: %d splits x %lld outputs x 4 bytes exceed the %u-byte static scratch\n",
                    eff, (long long)out_elems, (unsigned)XGEN_PATCONV_STATIC_SCRATCH_BYTES);
        return XGEN_ERR_SHAPE;
    }
    uint32_t *scratch = nullptr;
    {
        // First call on a device: resolve the device address of the array (in host code the
        // array's name is only a handle, not an address a kernel can use).
        std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
        scratch = g_static_scratch_addr[h->device];
        if (!scratch) {
            int prev = 0;
            if (cudaGetDevice(&prev) != cudaSuccess) return XGEN_ERR_CUDA;
            if (prev != h->device && cudaSetDevice(h->device) != cudaSuccess) return XGEN_ERR_CUDA;
            void *addr = nullptr;
            const cudaError_t e = cudaGetSymbolAddress(&addr, g_static_scratch);
            if (prev != h->device) cudaSetDevice(prev);
            if (log_cuda(e, "cudaGetSymbolAddress") != cudaSuccess || !addr) return XGEN_ERR_CUDA;
            scratch = g_static_scratch_addr[h->device] = static_cast<uint32_t *>(addr);
        }
    }
    const SplitChoice choice{eff, cps, scratch};
    return run_layer(h, x, n, hh, ww, bias, relu, y, stream, &choice);
}

xgen_status xgen_patconv_enqueue_host(const xgen_patconv_packed *h, const void *x, int32_t n, int32_t hh, int32_t ww,
                                      const void *bias, int32_t relu, void *y, void *stream) {
    if (!h || !x || !y) return XGEN_ERR_INVALID_ARG;
    if (n < 1 || hh < 1 || ww < 1) return XGEN_ERR_SHAPE;
    if (h->device < 0) return XGEN_ERR_CUDA;
    const PackedHost &p = h->host;
    const int ho = (hh + 2 - 3) / p.stride + 1, wo = (ww + 2 - 3) / p.stride + 1;
    const int xb = p.dtype == XGEN_F32 ? 4 : (p.dtype == XGEN_F16_F32ACC ? 2 : 1);
    const int yb = p.dtype == XGEN_F16_F32ACC ? 2 : 4;
    const size_t xbytes = (size_t)n * hh * ww * p.c_in * xb, ybytes = (size_t)n * ho * wo * p.c_out * yb;
    int prev = 0;
    if (cudaGetDevice(&prev) != cudaSuccess || cudaSetDevice(h->device) != cudaSuccess) return XGEN_ERR_CUDA;
    std::lock_guard<std::mutex> lock(h->host_mu);      // one host-buffer call per handle is enqueued at a time
    cudaStream_t st = (cudaStream_t)stream;
    xgen_status rs = XGEN_OK;
    cudaError_t e = cudaSuccess;
    if (xbytes > h->hx_bytes) {
        if (h->d_hx) cudaFree(h->d_hx);
        h->d_hx = nullptr; h->hx_bytes = 0;
        e = cudaMalloc(&h->d_hx, xbytes);
        if (e == cudaSuccess) h->hx_bytes = xbytes;
    }
    if (e == cudaSuccess && ybytes > h->hy_bytes) {
        if (h->d_hy) cudaFree(h->d_hy);
        h->d_hy = nullptr; h->hy_bytes = 0;
        e = cudaMalloc(&h->d_hy, ybytes);
        if (e == cudaSuccess) h->hy_bytes = ybytes;
    }
    if (e == cudaSuccess && bias && !h->d_hb) e = cudaMalloc(&h->d_hb, (size_t)p.c_out * 4);
    if (e != cudaSuccess) { rs = (e == cudaErrorMemoryAllocation) ? XGEN_ERR_ALLOC : XGEN_ERR_CUDA; cudaGetLastError(); }
    if (e == cudaSuccess && !h->s_in) e = cudaStreamCreateWithFlags(&h->s_in, cudaStreamNonBlocking);
    if (e == cudaSuccess && !h->s_out) e = cudaStreamCreateWithFlags(&h->s_out, cudaStreamNonBlocking);
    if (e == cudaSuccess && !h->ev_in) e = cudaEventCreateWithFlags(&h->ev_in, cudaEventDisableTiming);
    if (e == cudaSuccess && !h->ev_run) e = cudaEventCreateWithFlags(&h->ev_run, cudaEventDisableTiming);
    if (e == cudaSuccess && !h->ev_out) e = cudaEventCreateWithFlags(&h->ev_out, cudaEventDisableTiming);
    if (rs == XGEN_OK && e != cudaSuccess) { rs = XGEN_ERR_CUDA; cudaGetLastError(); }
    void *dx = h->d_hx, *dy = h->d_hy, *db = bias ? h->d_hb : nullptr;
    // Copy in on the handle's first stream, the layer on the caller's, copy out on the handle's
    // second stream: the caller's stream carries kernels only, so the copies of one handle
    // overlap the kernels and the copies (in the other direction) of other handles.
    if (rs == XGEN_OK) {
        if (h->host_call_before) {
            e = cudaStreamWaitEvent(h->s_in, h->ev_run, 0);           // the earlier call's kernel has read x and bias
            if (e == cudaSuccess) e = cudaStreamWaitEvent(st, h->ev_out, 0);   // and its copy out has read y
        }
        if (e == cudaSuccess) e = cudaMemcpyAsync(dx, x, xbytes, cudaMemcpyHostToDevice, h->s_in);
        if (e == cudaSuccess && bias) e = cudaMemcpyAsync(db, bias, (size_t)p.c_out * 4, cudaMemcpyHostToDevice, h->s_in);
        if (e == cudaSuccess) e = cudaEventRecord(h->ev_in, h->s_in);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(st, h->ev_in, 0);
        if (e != cudaSuccess) rs = XGEN_ERR_CUDA;
    }
    if (rs == XGEN_OK) rs = xgen_patconv_run(h, dx, n, hh, ww, db, relu, dy, stream);
    if (rs == XGEN_OK) {
        e = cudaEventRecord(h->ev_run, st);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(h->s_out, h->ev_run, 0);
        if (e == cudaSuccess) e = cudaMemcpyAsync(y, dy, ybytes, cudaMemcpyDeviceToHost, h->s_out);
        if (e == cudaSuccess) e = cudaEventRecord(h->ev_out, h->s_out);
        if (e != cudaSuccess) rs = XGEN_ERR_CUDA;
        h->host_call_before = true;
    }
    cudaSetDevice(prev);
    return rs;
}

xgen_status xgen_patconv_run_host(const xgen_patconv_packed *h, const void *x, int32_t n, int32_t hh, int32_t ww,
                                  const void *bias, int32_t relu, void *y) {
    xgen_status rs = xgen_patconv_enqueue_host(h, x, n, hh, ww, bias, relu, y, nullptr);
    if (rs != XGEN_OK) return rs;
    int prev = 0;
    if (cudaGetDevice(&prev) != cudaSuccess || cudaSetDevice(h->device) != cudaSuccess) return XGEN_ERR_CUDA;
    if (cudaStreamSynchronize(0) != cudaSuccess) rs = XGEN_ERR_CUDA;
    if (h->s_out && cudaStreamSynchronize(h->s_out) != cudaSuccess) rs = XGEN_ERR_CUDA;
    cudaSetDevice(prev);
    return rs;
}

}  // extern "C"
