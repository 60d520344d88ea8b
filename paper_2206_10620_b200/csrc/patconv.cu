// libpatconv: CUDA kernels (sm_100a) and the C ABI.
//
// One thread block = one tile of output pixels x one block of contiguous output
// channels.  Each warp owns a filter group (J filters); each lane owns a
// 4x4 block of output pixels (2x4 at stride 2; up to LN images side by side for
// small images).
// Per chunk of input channels the block stages (cp.async) the input tile with
// its halo into channel planes in shared memory -- the NHWC -> plane transpose
// happens in that copy -- together with the block's slice of the command
// stream.  Each warp then interprets its commands (core_gen.inc): LOAD brings
// the thread's activation patch of one channel into registers once, and every
// surviving kernel of the group on that channel reuses it (the paper's load
// redundancy elimination, Sec. 2.3); the running sums live in tensor memory,
// addressed by filter slot.  The epilogue adds bias, applies ReLU, converts and
// stores straight from tensor memory: a group is a run of consecutive output
// channels, so a thread writes 32 contiguous bytes per pixel (operator fusion,
// Sec. 2.2).
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
constexpr int kMaxWarps = 16;

struct KParams {
    const void *x; void *y; const void *bias;
    const uint32_t *slots; const int32_t *seg_off; const int32_t *slot_oc;
    int n, h, w, ho, wo, c_in, c_out;
    int relu;
    int J, wpc, cc, n_chunks;
    int lx_log, ly_log, ln_log;          // lanes along x, y and images: 2^.. each, product 32
    int tiles_x, tiles_y;
    int tin_w, tin_h;                    // staged tile extents, input pixels
    int pitch, img_stride, plane_stride; // words
    int raw_planes;                      // planes of one staged chunk (cc / channels per word)
    int act_stage_words, cmd_stage_words, stage_words;
    int n_stages;
    int exp_off_words;                   // offset of the expanded tile (f16 / i8) in shared memory
    int tmem_cols, cols_per_warp;
    int flush_chunks;                    // i8: chunks between folds of the fp32 partial sums
    int vec_in;                          // c_in is a multiple of the channels per staged word
    int vec_out;                         // widest aligned store of an 8-channel piece: 8 or 4 words, 0 = scalar
    int tab_off_words;                   // offset of the per-pixel staging table in shared memory
    int seg_off_words;                   // offset of the block's copy of the segment offsets
    int use_tma;                         // stage tiles with the tensor-memory-access unit (aligned channel counts)
    int mbar_off_words;                  // one 8-byte mbarrier per stage
    int box_bytes;                       // bytes one tensor copy delivers (the whole box, padding included)
    int *status;                         // device word: set to 1 if a bounded wait ran out
    int ptab_off_words;                  // offset of the output-pixel table (32 lanes x pixels per thread)
    int fold;                            // i8: keep int32 totals in a second row and fold periodically
    int chunks_per_split;                // grid.z splits the channel chunks; 0 = no split
    uint32_t *partial;                   // split runs: [split][n*ho*wo*c_out] raw fp32 / int32 sums
    size_t out_elems;                    // n*ho*wo*c_out
};

// ---- small PTX wrappers -----------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void cp_async4(uint32_t dst, const void *src, int src_bytes) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t ta, uint32_t (&r)[8]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(ta) : "memory");
}
__device__ __forceinline__ void tmem_ld2(uint32_t ta, uint32_t (&r)[2]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x2.b32 {%0,%1}, [%2];"
                 : "=r"(r[0]), "=r"(r[1]) : "r"(ta) : "memory");
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

// Stride-1 layers use the packed two-wide fp32 FMA unless built with -DPATCONV_F2=0.
#ifndef PATCONV_F2
#define PATCONV_F2 1
#endif
#if PATCONV_F2
#define PATCONV_S1(np) PATCONV_CORE_S1_NP##np##_F2
#else
#define PATCONV_S1(np) PATCONV_CORE_S1_NP##np##_F1
#endif

// Wait for an mbarrier phase with a bound: on expiry the block-wide abort flag and the
// device status word are set and every later wait returns at once, so the kernel still
// runs to its end (releasing tensor memory) with garbage results the host can detect.
__device__ __forceinline__ bool mbar_wait(uint32_t mbar, uint32_t parity, volatile int *abort_flag, int *status) {
    for (int it = 0; it < 400000; ++it) {
        uint32_t ok;
        asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n selp.u32 %0, 1, 0, p;\n}"
                     : "=r"(ok) : "r"(mbar), "r"(parity), "r"(2000u) : "memory");
        if (ok) return true;
        if (*abort_flag) return false;
    }
    *abort_flag = 1;
    if (status) atomicExch(status, 1);
    return false;
}

template <int STRIDE, int NP>
__device__ __forceinline__ void run_commands(uint32_t sp, uint32_t tbase, uint32_t plane_bytes,
                                             uint32_t pitch_bytes, uint32_t tmem_base) {
    if (STRIDE == 1) {
        if (NP == 4) PATCONV_S1(4)(sp, tbase, plane_bytes, pitch_bytes, tmem_base);
        else if (NP == 8) PATCONV_S1(8)(sp, tbase, plane_bytes, pitch_bytes, tmem_base);
        else if (NP == 12) PATCONV_S1(12)(sp, tbase, plane_bytes, pitch_bytes, tmem_base);
        else PATCONV_S1(126)(sp, tbase, plane_bytes, pitch_bytes, tmem_base);
    } else {
        if (NP == 4) PATCONV_CORE_S2_NP4_F1(sp, tbase, plane_bytes, pitch_bytes, tmem_base);
        else if (NP == 8) PATCONV_CORE_S2_NP8_F1(sp, tbase, plane_bytes, pitch_bytes, tmem_base);
        else if (NP == 12) PATCONV_CORE_S2_NP12_F1(sp, tbase, plane_bytes, pitch_bytes, tmem_base);
        else PATCONV_CORE_S2_NP126_F1(sp, tbase, plane_bytes, pitch_bytes, tmem_base);
    }
}

// Channels carried by one staged 32-bit word, and element sizes.
template <int DT> struct DTraits;
template <> struct DTraits<XGEN_F32> { static constexpr int E = 1, xbytes = 4, ybytes = 4; };
template <> struct DTraits<XGEN_F16_F32ACC> { static constexpr int E = 2, xbytes = 2, ybytes = 2; };
template <> struct DTraits<XGEN_I8_I32> { static constexpr int E = 4, xbytes = 1, ybytes = 4; };

// ---- the kernel -----------------------------------------------------------------
template <int DT, int STRIDE, int NP>
__global__ void __launch_bounds__(kMaxWarps * 32)
patconv_kernel(const KParams P, const __grid_constant__ CUtensorMap tmap) {
    extern __shared__ __align__(128) uint32_t smem[];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    __shared__ int soc_s[kMaxWarps * 16];           // original output channel of every filter slot of this block
    constexpr int E = DTraits<DT>::E;
    constexpr int XB = DTraits<DT>::xbytes;
    constexpr int BW = STRIDE == 1 ? 4 : 2, BH = 4;   // output pixels per thread: BW x BH
    constexpr int T = BW * BH;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nthreads = blockDim.x;
    const int b = blockIdx.y;
    int tile = blockIdx.x;
    const int tx = tile % P.tiles_x; tile /= P.tiles_x;
    const int ty = tile % P.tiles_y;
    const int tn = tile / P.tiles_y;
    const int LX = 1 << P.lx_log, LY = 1 << P.ly_log;
    const int l_x = lane & (LX - 1), l_y = (lane >> P.lx_log) & (LY - 1), l_n = lane >> (P.lx_log + P.ly_log);
    const int TW = BW * LX, TH = BH * LY;
    const int n0 = tn << P.ln_log;                   // first image of the tile
    const int gy0 = ty * TH * STRIDE - 1, gx0 = tx * TW * STRIDE - 1;   // input coords of tile (0,0)

    // --- tensor memory for the running sums --------------------------------------
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_base_s)), "r"((uint32_t)P.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }

    // --- staging -------------------------------------------------------------------
    const int RP = P.raw_planes;                      // power of two
    const int rp = tid & (RP - 1);
    const int pix_step = nthreads / RP;
    const int npix = (P.tin_w * P.tin_h) << P.ln_log;
    const int32_t *seg_g = P.seg_off + (size_t)b * P.n_chunks * (P.wpc + 1);
    int *seg = reinterpret_cast<int *>(smem + P.seg_off_words);   // this block's slice, copied once
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t mbar0 = smem_base + (uint32_t)P.mbar_off_words * 4u;
    if (tid == 0) {
        abort_s = 0;
        if (P.use_tma) {
            for (int st = 0; st < P.n_stages; ++st)
                asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(mbar0 + 8u * st) : "memory");
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
    }

    // Per-pixel staging table, built once: {element index of channel 0 of the input
    // pixel, or -1 outside the image; word offset of the pixel inside a plane}.
    int2 *tab = reinterpret_cast<int2 *>(smem + P.tab_off_words);
    for (int q = tid; q < npix; q += nthreads) {
        const int col = q % P.tin_w, t2 = q / P.tin_w;
        const int row = t2 % P.tin_h, im = t2 / P.tin_h;
        const int gy = gy0 + row, gx = gx0 + col, gn = n0 + im;
        const bool ok = gn < P.n && gy >= 0 && gy < P.h && gx >= 0 && gx < P.w;
        tab[q] = make_int2(ok ? ((gn * P.h + gy) * P.w + gx) * P.c_in : -1,
                           im * P.img_stride + row * P.pitch + col);
    }
    for (int i = tid; i < P.wpc * P.J; i += nthreads) soc_s[i] = P.slot_oc[(size_t)blockIdx.y * P.wpc * P.J + i];
    // Output-pixel table: linear pixel index of (pixel t of lane l), or -1 outside the output.
    int *ptab = reinterpret_cast<int *>(smem + P.ptab_off_words);
    for (int i = tid; i < 32 * T; i += nthreads) {
        const int t = i >> 5, l2 = i & 31;
        const int p_x = l2 & (LX - 1), p_y = (l2 >> P.lx_log) & (LY - 1), p_n = l2 >> (P.lx_log + P.ly_log);
        const int ox = tx * TW + p_x * BW + (t % BW), oy = ty * TH + p_y * BH + (t / BW), on = n0 + p_n;
        ptab[i] = (on < P.n && oy < P.ho && ox < P.wo) ? (on * P.ho + oy) * P.wo + ox : -1;
    }
    __syncthreads();

    const int c_begin = P.chunks_per_split ? (int)blockIdx.z * P.chunks_per_split : 0;
    const int c_end = P.chunks_per_split ? min(P.n_chunks, c_begin + P.chunks_per_split) : P.n_chunks;

    // Segment offsets of this block's chunks: read once, not on every chunk's critical path.
    for (int i = tid; i < (c_end - c_begin) * (P.wpc + 1); i += nthreads) seg[i] = seg_g[c_begin * (P.wpc + 1) + i];
    __syncthreads();

    const int q0 = tid / RP;
    auto stage_load = [&](int c) {
        if (P.use_tma) {
            // one thread hands the tile (a 4-D box of the NHWC tensor, zero-filled outside the
            // image) and the command segment to the copy engine; an mbarrier counts the bytes
            if (c < c_end && tid == 0) {
                const int stage = (c - c_begin) % P.n_stages;
                const uint32_t raw = smem_base + (uint32_t)(stage * P.stage_words) * 4u;
                const uint32_t cmd = raw + (uint32_t)P.act_stage_words * 4u;
                const uint32_t mbar = mbar0 + 8u * stage;
                const int s0 = seg[(c - c_begin) * (P.wpc + 1)], s1 = seg[(c - c_begin) * (P.wpc + 1) + P.wpc];
                const uint32_t cmd_bytes = (uint32_t)(s1 - s0 + 2) * (kSlotWords * 4u);
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(mbar), "r"((uint32_t)P.box_bytes + cmd_bytes) : "memory");
                asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
                             ::"r"(raw), "l"(&tmap), "r"(c * P.cc), "r"(gx0), "r"(gy0), "r"(n0), "r"(mbar) : "memory");
                asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                             ::"r"(cmd), "l"(P.slots + (size_t)s0 * kSlotWords), "r"(cmd_bytes), "r"(mbar) : "memory");
            }
            return;
        }
        if (c < c_end) {
            const int stage = (c - c_begin) % P.n_stages;
            const uint32_t act = smem_base + (uint32_t)(stage * P.stage_words) * 4u;
            // activations: one 32-bit word = E consecutive channels of one pixel
            const int ic = c * P.cc + rp * E;
            const bool ic_ok = ic < P.c_in;
            const uint32_t plane = act + (uint32_t)(rp * P.plane_stride) * 4u;
            const char *xc = (const char *)P.x + (size_t)(ic_ok ? ic : 0) * XB;
            if (E == 1 || P.vec_in) {
                auto copy1 = [&](const int2 t) {
                    const bool ok = ic_ok && t.x >= 0;
                    cp_async4(plane + (uint32_t)t.y * 4u, xc + (size_t)(ok ? t.x : 0) * XB, ok ? 4 : 0);
                };
                int q = q0;
                for (; q + 3 * pix_step < npix; q += 4 * pix_step) {      // four independent copies in flight
                    const int2 t0 = tab[q], t1 = tab[q + pix_step], t2 = tab[q + 2 * pix_step], t3 = tab[q + 3 * pix_step];
                    copy1(t0); copy1(t1); copy1(t2); copy1(t3);
                }
                for (; q < npix; q += pix_step) copy1(tab[q]);
            } else {
                // channel count not a multiple of E: assemble the word element by element
                for (int q = q0; q < npix; q += pix_step) {
                    const int2 t = tab[q];
                    const bool ok = ic_ok && t.x >= 0;
                    const char *src = xc + (size_t)(ok ? t.x : 0) * XB;
                    uint32_t word = 0;
                    if (ok) {
                        for (int k = 0; k < E; ++k) {
                            if (ic + k < P.c_in) {
                                if (XB == 2) word |= (uint32_t)((const uint16_t *)src)[k] << (16 * k);
                                else word |= (uint32_t)((const uint8_t *)src)[k] << (8 * k);
                            }
                        }
                    }
                    asm volatile("st.shared.b32 [%0], %1;" ::"r"(plane + (uint32_t)t.y * 4u), "r"(word) : "memory");
                }
            }
            // this block's commands for the chunk: one contiguous segment
            const int s0 = seg[(c - c_begin) * (P.wpc + 1)], s1 = seg[(c - c_begin) * (P.wpc + 1) + P.wpc];
            const uint32_t cmd = act + (uint32_t)P.act_stage_words * 4u;
            const uint4 *gsrc = reinterpret_cast<const uint4 *>(P.slots + (size_t)s0 * kSlotWords);
            const int n16 = (s1 - s0 + 2) * 2;          // two look-ahead slots beyond the segment
            for (int i = tid; i < n16; i += nthreads) cp_async16(cmd + (uint32_t)i * 16u, gsrc + i);
        }
        cp_async_commit();
    };

    for (int s = 0; s < P.n_stages - 1; ++s) stage_load(c_begin + s);

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_cta = tmem_base_s;
    const uint32_t tmem_warp = tmem_cta + (((uint32_t)(warp & 3) * 32u) << 16) + (uint32_t)((warp >> 2) * P.cols_per_warp);
    {
        const uint32_t z[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        for (int c = 0; c < P.cols_per_warp; c += 8) tmem_st8(tmem_warp + c, z);
        tmem_wait_st();
    }
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

    const uint32_t thr_off = (uint32_t)(l_n * P.img_stride + l_y * BH * STRIDE * P.pitch + l_x * BW * STRIDE) * 4u;
    const uint32_t plane_bytes = (uint32_t)P.plane_stride * 4u, pitch_bytes = (uint32_t)P.pitch * 4u;

    // --- main loop over channel chunks --------------------------------------------
    for (int c = c_begin; c < c_end; ++c) {
        const int stage = (c - c_begin) % P.n_stages;
        if (P.use_tma) {
            if (!abort_s) mbar_wait(mbar0 + 8u * stage, (uint32_t)(((c - c_begin) / P.n_stages) & 1), &abort_s, P.status);
        } else {
            if (P.n_stages == 2) cp_async_wait<0>(); else cp_async_wait<1>();
        }
        __syncthreads();                       // chunk c has landed; everyone is done with chunk c-1
        stage_load(c + P.n_stages - 1);
        const uint32_t act = smem_base + (uint32_t)(stage * P.stage_words) * 4u;
        uint32_t tile_base = act;
        if (P.use_tma) {
            // the copy engine delivered [pixel][channel]; spread it into fp32 channel planes
            float *ex = reinterpret_cast<float *>(smem + P.exp_off_words);
            const uint4 *raw = reinterpret_cast<const uint4 *>(smem + stage * P.stage_words);
            const int vec_per_pix = (P.cc * XB) >> 4;                  // 16-byte pieces per pixel: 1 or 2
            constexpr int EPV = 16 / XB;                               // elements per piece
            for (int i = tid; i < npix; i += nthreads) {
                float *dst = ex + tab[i].y;
                for (int h2 = 0; h2 < vec_per_pix; ++h2) {
                    const uint4 wd = raw[i * vec_per_pix + h2];
                    const uint32_t w4[4] = {wd.x, wd.y, wd.z, wd.w};
                    float *d2 = dst + (size_t)(h2 * EPV) * P.plane_stride;
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        if (DT == XGEN_F32) {
                            d2[k * P.plane_stride] = __uint_as_float(w4[k]);
                        } else if (DT == XGEN_F16_F32ACC) {
                            const __half2 h2v = *reinterpret_cast<const __half2 *>(&w4[k]);
                            d2[(2 * k) * P.plane_stride] = __low2float(h2v);
                            d2[(2 * k + 1) * P.plane_stride] = __high2float(h2v);
                        } else {
#pragma unroll
                            for (int bq = 0; bq < 4; ++bq) d2[(4 * k + bq) * P.plane_stride] = (float)((w4[k] >> (8 * bq)) & 0xFFu);
                        }
                    }
                }
            }
            __syncthreads();
            tile_base = smem_base + (uint32_t)P.exp_off_words * 4u;
        } else if (DT != XGEN_F32) {
            // widen the staged words to fp32 planes (exact for fp16 and for uint8)
            float *ex = reinterpret_cast<float *>(smem + P.exp_off_words);
            const int quads = P.plane_stride >> 2;             // plane_stride is a multiple of 4
            for (int r = 0; r < RP; ++r) {
                const uint4 *raw = reinterpret_cast<const uint4 *>(smem + stage * P.stage_words + r * P.plane_stride);
                for (int i = tid; i < quads; i += nthreads) {
                    const uint4 wd = raw[i];
                    const uint32_t w4[4] = {wd.x, wd.y, wd.z, wd.w};
                    if (DT == XGEN_F16_F32ACC) {
                        float lo[4], hi[4];
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const __half2 h2 = *reinterpret_cast<const __half2 *>(&w4[k]);
                            lo[k] = __low2float(h2); hi[k] = __high2float(h2);
                        }
                        reinterpret_cast<float4 *>(ex + (2 * r) * P.plane_stride)[i] = make_float4(lo[0], lo[1], lo[2], lo[3]);
                        reinterpret_cast<float4 *>(ex + (2 * r + 1) * P.plane_stride)[i] = make_float4(hi[0], hi[1], hi[2], hi[3]);
                    } else {
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            reinterpret_cast<float4 *>(ex + (4 * r + k) * P.plane_stride)[i] =
                                make_float4((float)((w4[0] >> (8 * k)) & 0xFFu), (float)((w4[1] >> (8 * k)) & 0xFFu),
                                            (float)((w4[2] >> (8 * k)) & 0xFFu), (float)((w4[3] >> (8 * k)) & 0xFFu));
                    }
                }
            }
            __syncthreads();
            tile_base = smem_base + (uint32_t)P.exp_off_words * 4u;
        }
        const int s0 = seg[(c - c_begin) * (P.wpc + 1)], sg = seg[(c - c_begin) * (P.wpc + 1) + warp];
        uint32_t sp = act + (uint32_t)P.act_stage_words * 4u + (uint32_t)(sg - s0) * 32u;
        run_commands<STRIDE, NP>(sp, tile_base + thr_off, plane_bytes, pitch_bytes, tmem_warp);
        if (DT == XGEN_I8_I32 && P.fold && ((c - c_begin + 1) % P.flush_chunks == 0)) fold_partial_sums();
    }
    cp_async_wait<0>();
    if (DT == XGEN_I8_I32) { if (P.fold) fold_partial_sums(); else sums_to_int(); }

    // --- epilogue: bias + ReLU + convert, straight from tensor memory to NHWC -------
    // A group is a run of J consecutive output channels, so for one pixel a thread holds
    // 8 adjacent channels per 8 filter slots: 32 bytes (16 for fp16) it can store as one
    // piece.  No shared memory, no block-wide barrier: every warp drains on its own.
    const int *soc = soc_s + warp * P.J;
    const uint32_t tmem_res = (DT == XGEN_I8_I32 && P.fold) ? tmem_int : tmem_warp;
    const int oc_base = soc[0];
    if (oc_base >= 0) {
        const int *pt = ptab + lane;
        uint32_t *const part = P.partial ? P.partial + (size_t)blockIdx.z * P.out_elems : nullptr;
        for (int j0 = 0; j0 < P.J; j0 += 8) {
            const int oc0 = oc_base + j0;
            if (oc0 >= P.c_out) break;
            const int nv = min(8, P.c_out - oc0);                 // valid channels of this piece
            uint32_t bb[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) bb[k] = (P.bias && !part && k < nv) ? ((const uint32_t *)P.bias)[oc0 + k] : 0u;
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
                    const int pidx = pt[(t0 + tt) * 32];
                    if (pidx < 0) continue;
                    const size_t o = (size_t)pidx * P.c_out + oc0;
                    uint32_t r[8];
                    if (part) {
#pragma unroll
                        for (int k = 0; k < 8; ++k) r[k] = v[k][tt];
                    } else if (DT == XGEN_I8_I32) {
#pragma unroll
                        for (int k = 0; k < 8; ++k) { int q = (int)v[k][tt] + (int)bb[k]; if (P.relu) q = max(q, 0); r[k] = (uint32_t)q; }
                    } else {
#pragma unroll
                        for (int k = 0; k < 8; ++k) { float q = __uint_as_float(v[k][tt]) + __uint_as_float(bb[k]); if (P.relu) q = fmaxf(q, 0.f); r[k] = __float_as_uint(q); }
                    }
                    if (part || DT != XGEN_F16_F32ACC) {
                        uint32_t *dst = (part ? part : (uint32_t *)P.y) + o;
                        if (nv == 8 && P.vec_out == 8) {
                            asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(dst), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]) : "memory");
                        } else if (nv == 8 && P.vec_out == 4) {
                            *reinterpret_cast<uint4 *>(dst) = make_uint4(r[0], r[1], r[2], r[3]);
                            *reinterpret_cast<uint4 *>(dst + 4) = make_uint4(r[4], r[5], r[6], r[7]);
                        } else {
#pragma unroll
                            for (int k = 0; k < 8; ++k) if (k < nv) dst[k] = r[k];
                        }
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

static inline int pixels_per_thread_x(int stride) { return stride == 1 ? 4 : 2; }
static inline int pixels_per_thread(int stride) { return 4 * pixels_per_thread_x(stride); }

struct Geometry {
    int lx_log, ly_log, ln_log, tiles_x, tiles_y, tiles_n;
    int tin_w, tin_h, pitch, img_stride, plane_stride;
};

// Worst bank multiplicity of the 128-bit patch-row load for a candidate pitch.
static int row_load_conflicts(int stride, int lx_log, int ly_log, int pitch, int img_stride) {
    const int LX = 1 << lx_log, LY = 1 << ly_log;
    const int bw = pixels_per_thread_x(stride);
    auto addr = [&](int lane) {
        int x = lane & (LX - 1), y = (lane >> lx_log) & (LY - 1), n = lane >> (lx_log + ly_log);
        return n * img_stride + y * 4 * stride * pitch + x * bw * stride;   // words
    };
    int worst = 0;
    for (int ph = 0; ph < 4; ++ph) {                      // 128-bit accesses: 8 lanes per wavefront
        int cnt[32] = {0};
        for (int l = 0; l < 8; ++l) {
            int a = addr(ph * 8 + l);
            for (int k = 0; k < 4; ++k) cnt[(a + k) & 31]++;
        }
        for (int i = 0; i < 32; ++i) worst = worst > cnt[i] ? worst : cnt[i];
    }
    return worst;
}

static Geometry choose_geometry(int n, int ho, int wo, int stride) {
    Geometry best{};
    double best_eff = -1.0;
    const int bw = pixels_per_thread_x(stride), bh = 4;
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
    best.tin_w = stride == 1 ? TW + 2 : 2 * TW + 1;
    best.tin_h = stride == 1 ? TH + 2 : 2 * TH + 1;
    const int align = 4;                                  // 16-byte aligned patch rows
    int p0 = (best.tin_w + align - 1) / align * align, best_p = p0, best_c = 1 << 30;
    for (int p = p0; p <= p0 + 8; p += align) {
        int c = row_load_conflicts(stride, best.lx_log, best.ly_log, p, best.tin_h * p);
        if (c < best_c) { best_c = c; best_p = p; }
    }
    best.pitch = best_p;
    best.img_stride = best.tin_h * best.pitch;
    int ps = LN * best.img_stride;
    while ((ps & 31) != 4) ++ps;                          // planes 4 banks apart: conflict-free staging writes
    best.plane_stride = ps;
    return best;
}

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
    uint32_t *d_partial = nullptr;
    size_t partial_bytes = 0;
    int *d_status = nullptr;            // set by a kernel whose bounded wait ran out
    // device staging buffers of xgen_patconv_run_host, kept between calls (grow only)
    mutable std::mutex host_mu;
    mutable void *d_hx = nullptr, *d_hy = nullptr, *d_hb = nullptr;
    mutable size_t hx_bytes = 0, hy_bytes = 0;
};

static void free_device_layout(xgen_patconv_packed *h) {
    if (h->d_slots) cudaFree(h->d_slots);
    if (h->d_seg_off) cudaFree(h->d_seg_off);
    if (h->d_slot_oc) cudaFree(h->d_slot_oc);
    if (h->d_status) cudaFree(h->d_status);
    h->d_slots = nullptr; h->d_seg_off = nullptr; h->d_slot_oc = nullptr; h->d_status = nullptr;
}

// Upload the host layout; the device must be current.
static xgen_status upload_layout(xgen_patconv_packed *h) {
    const PackedHost &p = h->host;
    free_device_layout(h);
    // two spare slots: harmless over-read room for 16-byte copies
    size_t sb = (p.slots.size() + 2 * kSlotWords) * 4, gb = p.seg_off.size() * 4, ob = p.slot_oc.size() * 4;
    cudaError_t e = cudaMalloc(&h->d_slots, sb);
    if (e == cudaSuccess) e = cudaMalloc(&h->d_seg_off, gb);
    if (e == cudaSuccess) e = cudaMalloc(&h->d_slot_oc, ob);
    if (e == cudaSuccess) e = cudaMalloc(&h->d_status, sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(h->d_status, 0, sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(h->d_slots, 0, sb);
    if (e == cudaSuccess) e = cudaMemcpy(h->d_slots, p.slots.data(), p.slots.size() * 4, cudaMemcpyHostToDevice);
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
    if (e != cudaSuccess && getenv("XGEN_PATCONV_LOG"))
        fprintf(stderr, "libpatconv: %s: %s\n", what, cudaGetErrorString(e));
    return e;
}

// cuTensorMapEncodeTiled, fetched through the runtime so the library does not link libcuda.
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    static std::mutex m;
    std::lock_guard<std::mutex> lock(m);
    if (!tried) {
        tried = true;
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)ptr;
        else
            cudaGetLastError();
    }
    return fn;
}

template <int DT, int STRIDE>
static cudaError_t launch_np(int np, dim3 grid, dim3 block, size_t smem, cudaStream_t st, const KParams &kp, const CUtensorMap &tm) {
    auto go = [&](auto kern) -> cudaError_t {
        // the opt-in to large dynamic shared memory is per function and per device: do it once
        static std::mutex mu;
        static std::vector<std::pair<const void *, int>> done;
        {
            std::lock_guard<std::mutex> lock(mu);
            int dev = 0;
            cudaGetDevice(&dev);
            const std::pair<const void *, int> key((const void *)kern, dev);
            bool found = false;
            for (const auto &k : done) found = found || k == key;
            if (!found) {
                cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemMaxDynamic);
                if (e != cudaSuccess) return log_cuda(e, "cudaFuncSetAttribute");
                done.push_back(key);
            }
        }
        kern<<<grid, block, smem, st>>>(kp, tm);
        return log_cuda(cudaGetLastError(), "kernel launch");
    };
    switch (np) {
        case 4: return go(patconv_kernel<DT, STRIDE, 4>);
        case 8: return go(patconv_kernel<DT, STRIDE, 8>);
        case 12: return go(patconv_kernel<DT, STRIDE, 12>);
        default: return go(patconv_kernel<DT, STRIDE, 126>);
    }
}

static int next_pow2(int v) { int p = 32; while (p < v) p <<= 1; return p; }

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
        PackConfig cfg = choose_pack_config(desc->c_in, desc->c_out, desc->dtype, desc->stride);
        if (const char *e = getenv("XGEN_PATCONV_J")) { int v = atoi(e); if (v == 4 || v == 8 || v == 16 || v == 32) {
            cfg.filters_per_group = v;
            int groups = (desc->c_out + v - 1) / v; cfg.groups_per_block = groups < kMaxWarps ? groups : kMaxWarps; } }
        if (const char *e = getenv("XGEN_PATCONV_WPC")) { int v = atoi(e); if (v >= 1 && v <= kMaxWarps) {
            int groups = (desc->c_out + cfg.filters_per_group - 1) / cfg.filters_per_group; cfg.groups_per_block = groups < v ? groups : v; } }
        if (const char *e = getenv("XGEN_PATCONV_CC")) { int v = atoi(e); if (v == 2 || v == 4 || v == 8 || v == 16) cfg.channels_per_chunk = v; }
        if (desc->dtype == XGEN_I8_I32 && cfg.channels_per_chunk < 4) cfg.channels_per_chunk = 4;
        st = pack_host(*desc, dense_w_host, pattern_id_host, cfg, h->host);
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
    if (h->d_hx) cudaFree(h->d_hx);
    if (h->d_hy) cudaFree(h->d_hy);
    if (h->d_hb) cudaFree(h->d_hb);
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

xgen_status xgen_patconv_plan(xgen_patconv_packed *h, int32_t n, int32_t hh, int32_t ww) {
    if (!h) return XGEN_ERR_INVALID_ARG;
    if (n < 1 || hh < 1 || ww < 1) return XGEN_ERR_SHAPE;
    if (h->device < 0) return XGEN_ERR_CUDA;
    const PackedHost &p = h->host;
    const int ho = (hh + 2 - 3) / p.stride + 1, wo = (ww + 2 - 3) / p.stride + 1;
    if ((int64_t)n * ho * wo * p.c_out > 0x7FFFFFFFLL) return XGEN_ERR_SHAPE;
    const Geometry g = choose_geometry(n, ho, wo, p.stride);
    const int64_t ctas = (int64_t)g.tiles_x * g.tiles_y * g.tiles_n * p.n_blocks;
    const int flush_chunks_plan = 16777216 / (p.cc * 4 * 32640);
    const int cols_per_warp = p.J * pixels_per_thread(p.stride) * ((p.dtype == XGEN_I8_I32 && p.n_chunks > flush_chunks_plan) ? 2 : 1);
    const int warp_slots = 4 * (512 / cols_per_warp);                 // per SM, set by tensor memory
    int sms = 148;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, h->device);
    const size_t out_bytes = (size_t)n * ho * wo * p.c_out * 4;
    // Pick the split count with a small cost model (microseconds): blocks run in waves of
    // (SMs x blocks per SM); a block costs a fixed prologue + epilogue plus its share of the
    // multiply-adds at the rate one busy SM sustains; a split adds one write and one read of
    // the fp32 output per part, plus a second launch.
    const double blocks_per_wave = (double)sms * (warp_slots / p.wpc > 0 ? warp_slots / p.wpc : 1);
    const double macs_per_block = 4.0 * (double)p.stats.kernels_surviving * (double)n * ho * wo / (double)ctas;
    const double t_work = macs_per_block / 72e3, t_fixed = 10.0;      // 72 GMAC/s per SM, 10 us
    auto estimate = [&](int64_t k) {
        const int cps_k = (int)((p.n_chunks + k - 1) / k);
        const int64_t parts = (p.n_chunks + cps_k - 1) / cps_k;
        const double waves = std::ceil((double)(ctas * parts) / blocks_per_wave);
        double t = waves * (t_fixed + t_work / (double)parts);
        if (parts > 1) t += 3.0 + ((double)parts * 2.0 + 1.0) * (double)out_bytes / 4e6;   // 4 TB/s
        return t;
    };
    int64_t splits = 1;
    double best_t = estimate(1);
    for (int64_t k = 2; k <= p.n_chunks; ++k) {
        const double t = estimate(k);
        if (t < 0.9 * best_t || (splits > 1 && t < best_t)) { best_t = t; splits = k; }
    }
    if (const char *e = getenv("XGEN_PATCONV_SPLIT")) { int v = atoi(e); if (v >= 1) splits = v < p.n_chunks ? v : p.n_chunks; }
    if (splits < 1) splits = 1;
    const int cps = (int)((p.n_chunks + splits - 1) / splits);
    splits = (p.n_chunks + cps - 1) / cps;
    int prev = 0;
    if (cudaGetDevice(&prev) != cudaSuccess || cudaSetDevice(h->device) != cudaSuccess) return XGEN_ERR_CUDA;
    xgen_status rs = XGEN_OK;
    if (cudaDeviceSynchronize() != cudaSuccess) rs = XGEN_ERR_CUDA;
    if (rs == XGEN_OK && splits > 1) {
        const size_t need = out_bytes * (size_t)splits;
        if (need > h->partial_bytes) {
            if (h->d_partial) cudaFree(h->d_partial);
            h->d_partial = nullptr; h->partial_bytes = 0;
            if (cudaMalloc(&h->d_partial, need) != cudaSuccess) { cudaGetLastError(); rs = XGEN_ERR_ALLOC; }
            else h->partial_bytes = need;
        }
    }
    cudaSetDevice(prev);
    if (rs != XGEN_OK) { h->plan_splits = 1; h->plan_n = 0; return rs; }
    h->plan_n = n; h->plan_h = hh; h->plan_w = ww;
    h->plan_splits = (int)splits; h->plan_cps = cps;
    return XGEN_OK;
}

xgen_status xgen_patconv_last_status(const xgen_patconv_packed *h, void *stream) {
    if (!h) return XGEN_ERR_INVALID_ARG;
    cudaError_t e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) return XGEN_ERR_CUDA;
    if (cudaGetLastError() != cudaSuccess) return XGEN_ERR_CUDA;
    if (h->d_status) {
        // a kernel whose bounded wait for a tile copy ran out leaves a mark here
        int flag = 0;
        if (cudaMemcpy(&flag, h->d_status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return XGEN_ERR_CUDA;
        if (flag) {
            cudaMemset(h->d_status, 0, sizeof(int));
            return XGEN_ERR_TIMEOUT;
        }
    }
    return XGEN_OK;
}

}  // extern "C"

// Where a run keeps the partial sums of a split, when the caller (not the plan) decides.
struct SplitChoice { int splits, chunks_per_split; uint32_t *partial; };

static xgen_status run_layer(const xgen_patconv_packed *h, const void *x, int32_t n, int32_t hh, int32_t ww,
                             const void *bias, int32_t relu, void *y, void *stream, const SplitChoice *forced) {
    if (!h || !x || !y) return XGEN_ERR_INVALID_ARG;
    if (((uintptr_t)x & 15) || ((uintptr_t)y & 15) || ((uintptr_t)bias & 15)) return XGEN_ERR_INVALID_ARG;
    if (n < 1 || hh < 1 || ww < 1) return XGEN_ERR_SHAPE;
    const PackedHost &p = h->host;
    if (h->device < 0) return XGEN_ERR_CUDA;
    const int ho = (hh + 2 - 3) / p.stride + 1, wo = (ww + 2 - 3) / p.stride + 1;
    if ((int64_t)n * hh * ww * p.c_in > 0x7FFFFFFFLL || (int64_t)n * ho * wo * p.c_out > 0x7FFFFFFFLL) return XGEN_ERR_SHAPE;
    {
        const char *xa = (const char *)x, *ya = (const char *)y;
        const int xb = p.dtype == XGEN_F32 ? 4 : (p.dtype == XGEN_F16_F32ACC ? 2 : 1);
        const int yb = p.dtype == XGEN_F16_F32ACC ? 2 : 4;
        const char *xe = xa + (size_t)n * hh * ww * p.c_in * xb, *ye = ya + (size_t)n * ho * wo * p.c_out * yb;
        if (xa < ye && ya < xe) return XGEN_ERR_INVALID_ARG;   // overlap
    }
    Geometry g = choose_geometry(n, ho, wo, p.stride);
    KParams kp{};
    kp.x = x; kp.y = y; kp.bias = bias;
    kp.slots = h->d_slots; kp.seg_off = h->d_seg_off; kp.slot_oc = h->d_slot_oc;
    kp.n = n; kp.h = hh; kp.w = ww; kp.ho = ho; kp.wo = wo; kp.c_in = p.c_in; kp.c_out = p.c_out;
    kp.relu = relu ? 1 : 0;
    kp.J = p.J; kp.wpc = p.wpc; kp.cc = p.cc; kp.n_chunks = p.n_chunks;
    kp.lx_log = g.lx_log; kp.ly_log = g.ly_log; kp.ln_log = g.ln_log;
    kp.tiles_x = g.tiles_x; kp.tiles_y = g.tiles_y;
    kp.tin_w = g.tin_w; kp.tin_h = g.tin_h;
    kp.pitch = g.pitch; kp.img_stride = g.img_stride; kp.plane_stride = g.plane_stride;
    const int E = p.dtype == XGEN_F32 ? 1 : (p.dtype == XGEN_F16_F32ACC ? 2 : 4);
    kp.raw_planes = p.cc / E;
    const int xb = p.dtype == XGEN_F32 ? 4 : (p.dtype == XGEN_F16_F32ACC ? 2 : 1);
    const int npix_box = (g.tin_w * g.tin_h) << g.ln_log;
    // The copy engine needs 16-byte multiples: the channel run of a chunk and every global stride.
    EncodeTiledFn encode = nullptr;
    kp.use_tma = ((p.cc * xb) % 16 == 0) && (((size_t)p.c_in * xb) % 16 == 0) && g.tin_w <= 256 && g.tin_h <= 256 &&
                 !getenv("XGEN_PATCONV_NO_TMA") && (encode = encode_tiled_fn()) != nullptr;
    CUtensorMap tm;
    memset(&tm, 0, sizeof(tm));
    if (kp.use_tma) {
        const cuuint64_t gdim[4] = {(cuuint64_t)p.c_in, (cuuint64_t)ww, (cuuint64_t)hh, (cuuint64_t)n};
        const cuuint64_t gstr[3] = {(cuuint64_t)p.c_in * xb, (cuuint64_t)ww * p.c_in * xb, (cuuint64_t)hh * ww * p.c_in * xb};
        const cuuint32_t box[4] = {(cuuint32_t)p.cc, (cuuint32_t)g.tin_w, (cuuint32_t)g.tin_h, (cuuint32_t)(1 << g.ln_log)};
        const cuuint32_t estr[4] = {1, 1, 1, 1};
        const CUtensorMapDataType dt = p.dtype == XGEN_F32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                                     : (p.dtype == XGEN_F16_F32ACC ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8);
        const CUresult cr = encode(&tm, dt, 4, const_cast<void *>(x), gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                   CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (cr != CUDA_SUCCESS) {          // fall back to thread-issued copies
            if (getenv("XGEN_PATCONV_LOG")) fprintf(stderr, "libpatconv: cuTensorMapEncodeTiled failed (%d)\n", (int)cr);
            kp.use_tma = 0;
            memset(&tm, 0, sizeof(tm));
        }
    }
    kp.box_bytes = npix_box * p.cc * xb;
    kp.cmd_stage_words = ((p.max_seg_slots + 2) * kSlotWords + 31) & ~31;
    kp.status = h->d_status;
    kp.vec_in = (p.c_in % E) == 0;
    // widest aligned store per 8-channel piece: 8 words (32-byte aligned rows), 4, or scalar
    kp.vec_out = ((p.c_out % 8) == 0 && ((uintptr_t)y & 31) == 0) ? 8 : ((p.c_out % 4) == 0 ? 4 : 0);
    const bool is_i8 = p.dtype == XGEN_I8_I32;
    const int T = pixels_per_thread(p.stride);
    kp.flush_chunks = 16777216 / (p.cc * 4 * 32640);
    if (kp.flush_chunks < 1) return XGEN_ERR_UNSUPPORTED;
    kp.fold = (is_i8 && p.n_chunks > kp.flush_chunks) ? 1 : 0;
    kp.cols_per_warp = p.J * T * (kp.fold ? 2 : 1);
    kp.tmem_cols = next_pow2(((p.wpc + 3) / 4) * kp.cols_per_warp);
    if (kp.tmem_cols > 512) return XGEN_ERR_UNSUPPORTED;
    int exp_words = 0;
    auto set_stage_layout = [&]() {
        kp.act_stage_words = kp.use_tma ? ((kp.box_bytes / 4 + 31) & ~31) : ((kp.raw_planes * g.plane_stride + 31) & ~31);
        kp.stage_words = kp.act_stage_words + kp.cmd_stage_words;
        exp_words = (p.dtype == XGEN_F32 && !kp.use_tma) ? 0 : ((p.cc * g.plane_stride + 31) & ~31);
    };
    set_stage_layout();
    const int npix_tile = (g.tin_w * g.tin_h) << g.ln_log;
    const int max_ctas = 512 / kp.tmem_cols;          // blocks per SM that tensor memory has columns for
    // Pick the stage count: three stages unless two let more blocks share an SM.
    const size_t seg_words = ((size_t)p.n_chunks * (p.wpc + 1) + 1) & ~(size_t)1;
    auto smem_words = [&](int stages) {
        size_t w = (size_t)stages * kp.stage_words + exp_words;
        return ((w + 1) & ~(size_t)1) + 2 * (size_t)npix_tile + 32 * (size_t)T + seg_words + 8;   // + mbarriers
    };
    auto occupancy = [&](size_t words) {
        int o = (int)((size_t)kSmemPerSM / (words * 4 + 2112));     // + static and per-block reserved shared memory
        return o < max_ctas ? o : max_ctas;
    };
    if (kp.use_tma && smem_words(2) * 4 > (size_t)kSmemMaxDynamic) {
        kp.use_tma = 0;                   // the copy engine's layout needs one more tile buffer: does not fit
        set_stage_layout();
    }
    int n_stages = 3;
    if (smem_words(3) * 4 > (size_t)kSmemMaxDynamic || occupancy(smem_words(2)) > occupancy(smem_words(3))) n_stages = 2;
    kp.n_stages = n_stages;
    kp.exp_off_words = n_stages * kp.stage_words;
    size_t words = smem_words(n_stages);
    kp.mbar_off_words = (int)(words - 8);
    kp.seg_off_words = kp.mbar_off_words - (int)seg_words;
    kp.ptab_off_words = kp.seg_off_words - 32 * T;
    kp.tab_off_words = kp.ptab_off_words - 2 * npix_tile;
    size_t smem = words * 4;
    const bool split = forced ? forced->splits > 1
                              : (h->plan_splits > 1 && h->plan_n == n && h->plan_h == hh && h->plan_w == ww && h->d_partial);
    const int n_splits = forced ? forced->splits : h->plan_splits;
    uint32_t *const partial = forced ? forced->partial : h->d_partial;
    kp.out_elems = (size_t)n * ho * wo * p.c_out;
    kp.chunks_per_split = split ? (forced ? forced->chunks_per_split : h->plan_cps) : 0;
    kp.partial = split ? partial : nullptr;
    // Never let more blocks share an SM than tensor memory has columns for.
    const size_t floor_bytes = (size_t)kSmemPerSM / (max_ctas + 1);
    if (smem < floor_bytes) smem = floor_bytes;
    if (smem > (size_t)kSmemMaxDynamic) return XGEN_ERR_UNSUPPORTED;

    int prev = 0;
    if (cudaGetDevice(&prev) != cudaSuccess) return XGEN_ERR_CUDA;
    if (prev != h->device && cudaSetDevice(h->device) != cudaSuccess) return XGEN_ERR_CUDA;
    dim3 grid((unsigned)(g.tiles_x * g.tiles_y * g.tiles_n), (unsigned)p.n_blocks, (unsigned)(split ? n_splits : 1)), block((unsigned)(p.wpc * 32), 1, 1);
    cudaStream_t st = (cudaStream_t)stream;
    cudaError_t e;
    if (p.dtype == XGEN_F32)
        e = p.stride == 1 ? launch_np<XGEN_F32, 1>(p.np, grid, block, smem, st, kp, tm) : launch_np<XGEN_F32, 2>(p.np, grid, block, smem, st, kp, tm);
    else if (p.dtype == XGEN_F16_F32ACC)
        e = p.stride == 1 ? launch_np<XGEN_F16_F32ACC, 1>(p.np, grid, block, smem, st, kp, tm) : launch_np<XGEN_F16_F32ACC, 2>(p.np, grid, block, smem, st, kp, tm);
    else
        e = p.stride == 1 ? launch_np<XGEN_I8_I32, 1>(p.np, grid, block, smem, st, kp, tm) : launch_np<XGEN_I8_I32, 2>(p.np, grid, block, smem, st, kp, tm);
    if (e == cudaSuccess && split) {
        const int vec = kp.vec_out >= 4 ? 1 : 0;
        const size_t items = vec ? kp.out_elems / 4 : kp.out_elems;
        const unsigned blocks = (unsigned)((items + 255) / 256);
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(blocks, 1, 1); cfg.blockDim = dim3(256, 1, 1); cfg.dynamicSmemBytes = 0; cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        const uint32_t *part_c = partial;
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

xgen_status xgen_patconv_run(const xgen_patconv_packed *h, const void *x, int32_t n, int32_t hh, int32_t ww,
                             const void *bias, int32_t relu, void *y, void *stream) {
    return run_layer(h, x, n, hh, ww, bias, relu, y, stream, nullptr);
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
        if (getenv("XGEN_PATCONV_LOG"))
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

xgen_status xgen_patconv_run_host(const xgen_patconv_packed *h, const void *x, int32_t n, int32_t hh, int32_t ww,
                                  const void *bias, int32_t relu, void *y) {
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
    std::lock_guard<std::mutex> lock(h->host_mu);      // one host-buffer call per handle at a time
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
    if (e != cudaSuccess) { rs = XGEN_ERR_ALLOC; cudaGetLastError(); }
    void *dx = h->d_hx, *dy = h->d_hy, *db = bias ? h->d_hb : nullptr;
    if (rs == XGEN_OK) {
        e = cudaMemcpyAsync(dx, x, xbytes, cudaMemcpyHostToDevice, 0);
        if (e == cudaSuccess && bias) e = cudaMemcpyAsync(db, bias, (size_t)p.c_out * 4, cudaMemcpyHostToDevice, 0);
        if (e != cudaSuccess) rs = XGEN_ERR_CUDA;
    }
    if (rs == XGEN_OK) rs = xgen_patconv_run(h, dx, n, hh, ww, db, relu, dy, nullptr);
    if (rs == XGEN_OK) {
        e = cudaMemcpyAsync(y, dy, ybytes, cudaMemcpyDeviceToHost, 0);
        if (e == cudaSuccess) e = cudaStreamSynchronize(0);
        if (e != cudaSuccess) rs = XGEN_ERR_CUDA;
    }
    cudaSetDevice(prev);
    return rs;
}

}  // extern "C"
