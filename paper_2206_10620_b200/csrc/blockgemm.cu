// libpatconv: block-pruned matrix product (paper Sec. 2.1, "Block-Based Pruning") for
// sm_100a, and its C ABI.
//
// y[m][oc] = act(bias[oc] + sum over the kept entries of row oc of W[oc][c] * x[m][c]).
// Inside a pruning block whole rows and whole columns are gone, so what is left of a block
// is a small dense matrix on a subset of the input columns and a subset of the output
// channels -- subsets that differ from block to block.  Both selections are data:
//
//  * the kept COLUMNS select which activations a thread needs.  A thread block stages a tile
//    of 256 rows of x for a slice of the input columns in shared memory (asynchronous copies,
//    two stages), and a warp reads from it only the columns its commands name;
//  * the kept ROWS select which running sums a multiply-add goes to.  Registers cannot be
//    indexed at run time, tensor-memory columns can: every warp keeps the sums of its 16
//    output channels x 8 rows of x per lane in 128 tensor-memory columns, and a command
//    fetches the row it addresses, adds 8 columns x 8 rows of x to it with two-wide fp32
//    FMAs, and puts it back.
//
// A row command is three 16-byte units (header, weights 0..3, weights 4..7); gen_blockgemm.py
// holds the code that interprets them.
//
// The packer turns every (warp, stage) into a list of column groups (up to eight kept columns
// of one pruning block, padded with a column that reads zeros) each followed by one command
// per kept row with the eight weights.  Pruned rows and columns cost nothing at run time.
//
// No tensor-core instruction is used: fp32 data has no exact tensor-core path, and the
// selection of columns would have to be gathered into operand tiles first.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "blockgemm.h"
#include "blockgemm_core.inc"
#include "patconv_internal.h"

namespace blockgemm {

constexpr int kRowsPerWarp = 16;       // output channels a warp accumulates
constexpr int kPixPerLane = 8;         // rows of x a lane owns: lane, lane + 32, ...
constexpr int kTileM = 32 * kPixPerLane;
constexpr int kMaxWarps = 16;
constexpr int kDefaultWarps = 8;       // two such thread blocks share an SM and overlap their phases
constexpr int kGroupCols = 8;          // columns of one activation load
constexpr int kSmemLimit = 220 * 1024;

struct Host {
    int k = 0, c_out = 0, br = 0, bc = 0;
    xgen_dtype dtype = XGEN_F32;
    int warps = 0, rows_per_block = 0, n_rb = 0, ks = 0, ns = 0;
    int max_stage_units = 0;
    std::vector<uint32_t> stream;       // 4 words per 16-byte unit
    std::vector<int32_t> seg_off;       // [(rb * ns + s) * (warps + 1) + w], in units
    xgen_blockgemm_stats stats{};
};

}  // namespace blockgemm

struct xgen_blockgemm_packed {
    blockgemm::Host host;
    int device = -1;
    uint32_t *d_stream = nullptr;
    int32_t *d_seg = nullptr;
    std::atomic<bool> attr_set{false};
};

namespace blockgemm {

static float half_to_float(uint16_t h) {
    const uint32_t sign = (uint32_t)(h >> 15) << 31;
    int exp = (h >> 10) & 0x1f;
    uint32_t man = h & 0x3ff;
    uint32_t bits;
    if (exp == 0) {
        if (man == 0) bits = sign;
        else {
            int e = -1;
            do { ++e; man <<= 1; } while (!(man & 0x400));
            bits = sign | (uint32_t)(127 - 15 - e) << 23 | (man & 0x3ff) << 13;
        }
    } else if (exp == 31) bits = sign | 0x7f800000u | man << 13;
    else bits = sign | (uint32_t)(exp - 15 + 127) << 23 | man << 13;
    float f;
    std::memcpy(&f, &bits, 4);
    return f;
}

// Build the stream for a given number of staged columns.  Returns false if nothing fits.
static void build_stream(Host &h, const std::vector<float> &w, const uint8_t *row_keep, const uint8_t *col_keep, int ks) {
    const int nbc = (h.k + h.bc - 1) / h.bc;
    h.ks = ks;
    h.ns = (h.k + ks - 1) / ks;
    h.stream.clear();
    h.seg_off.assign((size_t)h.n_rb * h.ns * (h.warps + 1), 0);
    h.max_stage_units = 0;
    int64_t padded = 0, groups = 0, row_cmds = 0;
    std::vector<int> rows, cols, pend_rows, pend_cols;
    auto flush = [&](int r0, int c0) {
        if (pend_rows.empty() || pend_cols.empty()) { pend_rows.clear(); pend_cols.clear(); return; }
        for (size_t g = 0; g < pend_cols.size(); g += kGroupCols) {
            const int nc = (int)std::min<size_t>(kGroupCols, pend_cols.size() - g);
            uint32_t idx[2] = {0, 0};
            for (int i = 0; i < kGroupCols; ++i) {
                const uint32_t ci = i < nc ? (uint32_t)(pend_cols[g + i] - c0) : (uint32_t)ks;   // ks = the column of zeros
                idx[i / 4] |= ci << (8 * (i % 4));
            }
            h.stream.push_back((uint32_t)pend_rows.size());
            h.stream.push_back(idx[0]);
            h.stream.push_back(idx[1]);
            h.stream.push_back(0);
            ++groups;
            for (int r : pend_rows) {
                h.stream.push_back((uint32_t)((r - r0) * kPixPerLane));
                h.stream.push_back(0); h.stream.push_back(0); h.stream.push_back(0);
                for (int i = 0; i < kGroupCols; ++i) {
                    float v = 0.0f;
                    if (i < nc) v = w[(size_t)r * h.k + pend_cols[g + i]]; else ++padded;
                    uint32_t bits;
                    std::memcpy(&bits, &v, 4);
                    h.stream.push_back(bits);
                }
                ++row_cmds;
            }
        }
        pend_rows.clear();
        pend_cols.clear();
    };
    for (int rb = 0; rb < h.n_rb; ++rb) {
        for (int s = 0; s < h.ns; ++s) {
            const size_t seg_base = ((size_t)rb * h.ns + s) * (h.warps + 1);
            const size_t stage_start = h.stream.size() / 4;
            for (int wi = 0; wi < h.warps; ++wi) {
                h.seg_off[seg_base + wi] = (int32_t)(h.stream.size() / 4);
                const int r0 = rb * h.rows_per_block + wi * kRowsPerWarp;
                const int r1 = std::min(r0 + kRowsPerWarp, h.c_out);
                const int c0 = s * ks, c1 = std::min(c0 + ks, h.k);
                if (r0 >= r1) continue;
                for (int i = r0 / h.br; i <= (r1 - 1) / h.br; ++i) {
                    for (int j = c0 / h.bc; j <= (c1 - 1) / h.bc; ++j) {
                        const size_t blk = (size_t)i * nbc + j;
                        rows.clear(); cols.clear();
                        for (int r = std::max(r0, i * h.br); r < std::min(r1, (i + 1) * h.br); ++r)
                            if (row_keep[blk * h.br + (r - i * h.br)]) rows.push_back(r);
                        for (int c = std::max(c0, j * h.bc); c < std::min(c1, (j + 1) * h.bc); ++c)
                            if (col_keep[blk * h.bc + (c - j * h.bc)]) cols.push_back(c);
                        if (rows.empty() || cols.empty()) continue;
                        // neighbouring blocks with the same kept rows share column groups
                        if (!pend_rows.empty() && rows != pend_rows) flush(r0, c0);
                        if (pend_rows.empty()) pend_rows = rows;
                        pend_cols.insert(pend_cols.end(), cols.begin(), cols.end());
                    }
                    flush(r0, c0);
                }
            }
            h.seg_off[seg_base + h.warps] = (int32_t)(h.stream.size() / 4);
            h.max_stage_units = std::max(h.max_stage_units, (int)(h.stream.size() / 4 - stage_start));
        }
    }
    h.stats.padded_slots = padded;
    h.stats.column_groups = groups;
    h.stats.row_commands = row_cmds;
}

static size_t raw_pitch_words(xgen_dtype dt, int ks) {
    // one row of x of a stage plus the column of zeros; an odd number of 32-bit words, so that
    // the lanes of a warp (consecutive rows of x) read distinct banks
    return dt == XGEN_F32 ? (size_t)ks + 1 : (size_t)ks / 2 + 1;
}

static size_t smem_bytes(const Host &h) {
    return 2 * (size_t)kTileM * raw_pitch_words(h.dtype, h.ks) * 4 + 2 * (size_t)(h.max_stage_units + 1) * 16;   // + 1: the look-ahead of the last command
}

struct GParams {
    const void *x; void *y; const float *bias;
    const uint4 *stream; const int32_t *seg_off;
    long long m;
    int k, c_out;
    int warps, rows_per_block, n_rb, ks, ns;
    int relu;
    int async_x;            // rows of x can be copied asynchronously, 4 bytes at a time
    int vec_y;              // a warp's 16 channels of a row of y can be stored 16 bytes at a time
    int cmd_units;          // 16-byte units of one command buffer
    int tmem_cols;
};

// ---- PTX wrappers -----------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
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
__device__ __forceinline__ unsigned long long pack2(uint32_t lo, uint32_t hi) {
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(unsigned long long v, uint32_t &lo, uint32_t &hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(v));
}
__device__ __forceinline__ unsigned long long fma2(unsigned long long a, unsigned long long b, unsigned long long c) {
    unsigned long long d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ void cp_async4(uint32_t dst, const void *src, int src_bytes) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

// One thread block = 256 rows of x (a lane owns rows lane, lane + 32, ... of the tile) x one
// block of up to 256 output channels (16 per warp).
template <int DT, int KS>
__global__ void __launch_bounds__(kMaxWarps * 32, 1) blockgemm_kernel(const GParams P) {
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ uint32_t tmem_base_s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nthreads = P.warps * 32;
    const int rb = (int)(blockIdx.x % (unsigned)P.n_rb);
    const long long tile = blockIdx.x / (unsigned)P.n_rb;
    const long long m0 = tile * kTileM;
    constexpr int pitch = DT == XGEN_F32 ? KS + 1 : KS / 2 + 1;    // words per staged row of x
    constexpr int ks_log = KS == 32 ? 5 : KS == 16 ? 4 : 3;
    uint32_t *raw = reinterpret_cast<uint32_t *>(smem);                                   // [2][kTileM][pitch]
    uint4 *cmd = reinterpret_cast<uint4 *>(smem + 2 * (size_t)kTileM * pitch * 4);        // [2][cmd_units]

    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_base_s)), "r"((uint32_t)P.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // the column of zeros behind every staged row (padding slots of a column group read it)
    for (int i = tid; i < 2 * kTileM; i += nthreads) {
        raw[(size_t)i * pitch + pitch - 1] = 0u;
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_cta = tmem_base_s;
    const uint32_t tw = tmem_cta + (((uint32_t)(warp & 3) * 32u) << 16) + (uint32_t)((warp >> 2) * (kRowsPerWarp * kPixPerLane));
    {
        const uint32_t z[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#pragma unroll
        for (int c = 0; c < kRowsPerWarp * kPixPerLane; c += 8) tmem_st8(tw + c, z);
        tmem_wait_st();
    }

    const int32_t *seg_g = P.seg_off + (size_t)rb * P.ns * (P.warps + 1);

    // Stage s: copy the tile's rows of x for columns [s*ks, s*ks + ks) and the block's commands.
    // Where a stage's commands lie: the whole block's piece and this warp's part of it.
    auto load_seg = [&](int s, int &seg_b, int &seg_e, int &my_b, int &my_e) {
        if (s < P.ns) {
            const int32_t *sg = seg_g + (size_t)s * (P.warps + 1);
            seg_b = sg[0]; seg_e = sg[P.warps];
            my_b = sg[warp] - seg_b;
            my_e = sg[warp + 1] - seg_b;
        }
    };
    // Asynchronous staging, 4 bytes per copy: a thread always copies the same 4-byte unit of a row,
    // for rows rows_step apart, so its addresses advance by constants.
    constexpr int kUnits = DT == XGEN_F32 ? KS : KS / 2;          // 4-byte units of a staged row
    constexpr int kUnitElems = DT == XGEN_F32 ? 1 : 2;
    const int esz = DT == XGEN_F32 ? 4 : 2;
    const int a_row0 = tid / kUnits, a_unit = tid % kUnits;
    const int rows_step = nthreads / kUnits;
    const int a_iters = (kTileM + rows_step - 1) / rows_step;
    const long long a_left = min(P.m - m0, (long long)kTileM) - a_row0;   // rows of the tile from this thread's first row on
    const int a_lim = a_left <= 0 ? 0 : (int)min((long long)a_iters, (a_left + rows_step - 1) / rows_step);
    const char *a_src0 = static_cast<const char *>(P.x) + ((size_t)(m0 + a_row0) * P.k + (size_t)a_unit * kUnitElems) * esz;
    const size_t a_src_step = (size_t)rows_step * P.k * esz;
    const uint32_t a_dst0 = smem_u32(raw) + (uint32_t)(a_row0 * pitch + a_unit) * 4u;
    const uint32_t a_dst_step = (uint32_t)(rows_step * pitch) * 4u;

    auto issue = [&](int s, int buf, int seg_b, int seg_e) {
        uint4 *cdst = cmd + (size_t)buf * P.cmd_units;
        for (int u = tid; u < seg_e - seg_b; u += nthreads) cp_async16(smem_u32(cdst + u), P.stream + seg_b + u);
        uint32_t *rdst = raw + (size_t)buf * kTileM * pitch;
        const int c0 = s * KS;
        if (P.async_x) {
            const bool col_ok = c0 + a_unit * kUnitElems < P.k;
            const char *src = a_src0 + (size_t)c0 * esz;
            uint32_t dst = a_dst0 + (uint32_t)buf * (uint32_t)(kTileM * pitch * 4);
#pragma unroll 4
            for (int i = 0; i < a_iters; ++i) {
                const bool ok = col_ok && i < a_lim;
                if (a_row0 + i * rows_step < kTileM)     // (a tile's rows need not divide among the threads)
                    cp_async4(dst, ok ? (const void *)src : P.x, ok ? 4 : 0);
                src += a_src_step;
                dst += a_dst_step;
            }
        } else if (DT == XGEN_F32) {
            const float *x = static_cast<const float *>(P.x);
            constexpr int total = kTileM * KS;
            for (int e = tid; e < total; e += nthreads) {
                const int p = e >> ks_log, c = e & (KS - 1);
                const bool ok = (m0 + p < P.m) && (c0 + c < P.k);
                rdst[(size_t)p * pitch + c] = ok ? __float_as_uint(x[(size_t)(m0 + p) * P.k + c0 + c]) : 0u;
            }
        } else {
            const __half *x = static_cast<const __half *>(P.x);
            unsigned short *rh = reinterpret_cast<unsigned short *>(rdst);
            constexpr int total = kTileM * KS;
            for (int e = tid; e < total; e += nthreads) {
                const int p = e >> ks_log, c = e & (KS - 1);
                const bool ok = (m0 + p < P.m) && (c0 + c < P.k);
                rh[(size_t)p * pitch * 2 + c] = ok ? __half_as_ushort(x[(size_t)(m0 + p) * P.k + c0 + c]) : (unsigned short)0;
            }
        }
        cp_async_commit();
    };

    // The offsets of a stage are fetched one iteration before its copies are issued, so that
    // their latency is not waited for.
    int sb = 0, se = 0, nb = 0, ne = 0, sb2 = 0, se2 = 0, nb2 = 0, ne2 = 0;
    load_seg(0, sb, se, nb, ne);
    load_seg(1, sb2, se2, nb2, ne2);
    issue(0, 0, sb, se);
    for (int s = 0; s < P.ns; ++s) {
        const int buf = s & 1;
        const int my_b = nb, my_e = ne;
        cp_async_wait_all();
        __syncthreads();                 // stage s has landed; everybody has left stage s - 1
        if (s + 1 < P.ns) {
            issue(s + 1, buf ^ 1, sb2, se2);
            nb = nb2; ne = ne2;
            load_seg(s + 2, sb2, se2, nb2, ne2);
        }

        // The warp's commands of this stage, interpreted by the generated code (gen_blockgemm.py).
        uint32_t cp = smem_u32(cmd + (size_t)buf * P.cmd_units + my_b);
        const uint32_t ce = smem_u32(cmd + (size_t)buf * P.cmd_units + my_e);
        const uint32_t xbase = smem_u32(raw + (size_t)buf * kTileM * pitch + (size_t)lane * pitch);
        if (DT == XGEN_F32) {
            if (KS == 32) BLOCKGEMM_CORE_F32_KS32(cp, ce, xbase, tw);
            else if (KS == 16) BLOCKGEMM_CORE_F32_KS16(cp, ce, xbase, tw);
            else BLOCKGEMM_CORE_F32_KS8(cp, ce, xbase, tw);
        } else {
            if (KS == 32) BLOCKGEMM_CORE_F16_KS32(cp, ce, xbase, tw);
            else if (KS == 16) BLOCKGEMM_CORE_F16_KS16(cp, ce, xbase, tw);
            else BLOCKGEMM_CORE_F16_KS8(cp, ce, xbase, tw);
        }
    }
    tmem_wait_st();

    // Epilogue: bias, activation, conversion; a lane stores the warp's 16 channels of one row
    // of y at a time (64 contiguous bytes in fp32).
    const int oc0 = rb * P.rows_per_block + warp * kRowsPerWarp;
    if (oc0 < P.c_out) {
        const int n_oc = min(kRowsPerWarp, P.c_out - oc0);
        float bias[kRowsPerWarp];
#pragma unroll
        for (int r = 0; r < kRowsPerWarp; ++r) bias[r] = (P.bias && r < n_oc) ? P.bias[oc0 + r] : 0.0f;
#pragma unroll 1
        for (int hf = 0; hf < 2; ++hf) {
            uint32_t v[kRowsPerWarp][4];
#pragma unroll
            for (int r = 0; r < kRowsPerWarp; ++r) tmem_ld4(tw + r * kPixPerLane + 4 * hf, v[r]);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const long long p = m0 + lane + 32 * (4 * hf + j);
                if (p >= P.m) continue;
                float o[kRowsPerWarp];
#pragma unroll
                for (int r = 0; r < kRowsPerWarp; ++r) {
                    o[r] = __uint_as_float(v[r][j]) + bias[r];
                    if (P.relu) o[r] = fmaxf(o[r], 0.0f);
                }
                if (DT == XGEN_F32) {
                    float *y = static_cast<float *>(P.y) + (size_t)p * P.c_out + oc0;
                    if (P.vec_y && n_oc == kRowsPerWarp) {
#pragma unroll
                        for (int q = 0; q < 4; ++q)
                            reinterpret_cast<float4 *>(y)[q] = make_float4(o[4 * q], o[4 * q + 1], o[4 * q + 2], o[4 * q + 3]);
                    } else {
#pragma unroll
                        for (int r = 0; r < kRowsPerWarp; ++r) if (r < n_oc) y[r] = o[r];
                    }
                } else {
                    __half *y = static_cast<__half *>(P.y) + (size_t)p * P.c_out + oc0;
                    if (P.vec_y && n_oc == kRowsPerWarp) {
#pragma unroll
                        for (int q = 0; q < 2; ++q) {
                            uint4 pk;
                            __half2 h0 = __floats2half2_rn(o[8 * q], o[8 * q + 1]), h1 = __floats2half2_rn(o[8 * q + 2], o[8 * q + 3]);
                            __half2 h2 = __floats2half2_rn(o[8 * q + 4], o[8 * q + 5]), h3 = __floats2half2_rn(o[8 * q + 6], o[8 * q + 7]);
                            pk.x = *reinterpret_cast<uint32_t *>(&h0); pk.y = *reinterpret_cast<uint32_t *>(&h1);
                            pk.z = *reinterpret_cast<uint32_t *>(&h2); pk.w = *reinterpret_cast<uint32_t *>(&h3);
                            reinterpret_cast<uint4 *>(y)[q] = pk;
                        }
                    } else {
#pragma unroll
                        for (int r = 0; r < kRowsPerWarp; ++r) if (r < n_oc) y[r] = __float2half_rn(o[r]);
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

static const void *kernel_for(xgen_dtype dt, int ks) {
    if (dt == XGEN_F32)
        return ks == 32 ? (const void *)blockgemm_kernel<XGEN_F32, 32> : ks == 16 ? (const void *)blockgemm_kernel<XGEN_F32, 16>
                                                                                   : (const void *)blockgemm_kernel<XGEN_F32, 8>;
    return ks == 32 ? (const void *)blockgemm_kernel<XGEN_F16_F32ACC, 32> : ks == 16 ? (const void *)blockgemm_kernel<XGEN_F16_F32ACC, 16>
                                                                                      : (const void *)blockgemm_kernel<XGEN_F16_F32ACC, 8>;
}

}  // namespace blockgemm

using namespace blockgemm;

extern "C" {

xgen_status xgen_blockgemm_pack(const xgen_blockgemm_desc *d, const void *dense_w, const uint8_t *row_keep,
                                const uint8_t *col_keep, int device, xgen_blockgemm_packed **out) {
    if (!d || !dense_w || !row_keep || !col_keep || !out) return XGEN_ERR_INVALID_ARG;
    *out = nullptr;
    if (d->k < 1 || d->c_out < 1 || d->block_rows < 1 || d->block_cols < 1) return XGEN_ERR_INVALID_ARG;
    if (d->dtype != XGEN_F32 && d->dtype != XGEN_F16_F32ACC) return XGEN_ERR_UNSUPPORTED;
    if (d->warps_per_block < 0 || d->warps_per_block > kMaxWarps) return XGEN_ERR_INVALID_ARG;
    if ((int64_t)d->k * d->c_out > (int64_t)1 << 28) return XGEN_ERR_SHAPE;
    xgen_blockgemm_packed *h = new (std::nothrow) xgen_blockgemm_packed();
    if (!h) return XGEN_ERR_ALLOC;
    Host &H = h->host;
    try {
        H.k = d->k; H.c_out = d->c_out; H.br = d->block_rows; H.bc = d->block_cols; H.dtype = d->dtype;
        const int groups = (d->c_out + kRowsPerWarp - 1) / kRowsPerWarp;
        H.warps = std::min(groups, d->warps_per_block > 0 ? d->warps_per_block : kDefaultWarps);
        H.rows_per_block = H.warps * kRowsPerWarp;
        H.n_rb = (d->c_out + H.rows_per_block - 1) / H.rows_per_block;
        std::vector<float> w((size_t)d->k * d->c_out);
        if (d->dtype == XGEN_F32) std::memcpy(w.data(), dense_w, w.size() * 4);
        else for (size_t i = 0; i < w.size(); ++i) w[i] = half_to_float(static_cast<const uint16_t *>(dense_w)[i]);
        int ks = 32;
        while (ks > 8 && ks / 2 >= d->k) ks /= 2;
        for (;;) {
            build_stream(H, w, row_keep, col_keep, ks);
            if (smem_bytes(H) <= (size_t)kSmemLimit || ks == 8) break;
            ks /= 2;
        }
        if (smem_bytes(H) > (size_t)kSmemLimit) { delete h; return XGEN_ERR_SHAPE; }
        const int nbc = (d->k + d->block_cols - 1) / d->block_cols, nbr = (d->c_out + d->block_rows - 1) / d->block_rows;
        int64_t kept = 0;
        for (int i = 0; i < nbr; ++i)
            for (int j = 0; j < nbc; ++j) {
                const size_t blk = (size_t)i * nbc + j;
                int nr = 0, nc = 0;
                for (int r = 0; r < d->block_rows && i * d->block_rows + r < d->c_out; ++r) nr += row_keep[blk * d->block_rows + r] ? 1 : 0;
                for (int c = 0; c < d->block_cols && j * d->block_cols + c < d->k; ++c) nc += col_keep[blk * d->block_cols + c] ? 1 : 0;
                kept += (int64_t)nr * nc;
            }
        H.stats.weights_total = (int64_t)d->k * d->c_out;
        H.stats.weights_kept = kept;
        H.stats.weight_bytes = kept * (d->dtype == XGEN_F32 ? 4 : 2);
        H.stats.stream_bytes = (int64_t)H.stream.size() * 4 + (int64_t)H.seg_off.size() * 4;
        H.stats.rows_per_warp = kRowsPerWarp;
        H.stats.warps_per_block = H.warps;
        H.stats.row_blocks = H.n_rb;
        H.stats.stage_cols = H.ks;
        H.stats.n_stages = H.ns;
        H.stats.max_stage_bytes = H.max_stage_units * 16;
    } catch (const std::bad_alloc &) {
        delete h;
        return XGEN_ERR_ALLOC;
    }
    h->device = device;
    if (device >= 0) {
        int prev = 0;
        cudaGetDevice(&prev);
        xgen_status st = XGEN_OK;
        if (cudaSetDevice(device) != cudaSuccess) st = XGEN_ERR_CUDA;
        const size_t sb = std::max<size_t>(H.stream.size() * 4, 16), gb = H.seg_off.size() * 4;
        if (st == XGEN_OK && (cudaMalloc(&h->d_stream, sb) != cudaSuccess || cudaMalloc(&h->d_seg, gb) != cudaSuccess)) st = XGEN_ERR_ALLOC;
        if (st == XGEN_OK && ((!H.stream.empty() && cudaMemcpy(h->d_stream, H.stream.data(), H.stream.size() * 4, cudaMemcpyHostToDevice) != cudaSuccess) ||
                              cudaMemcpy(h->d_seg, H.seg_off.data(), gb, cudaMemcpyHostToDevice) != cudaSuccess)) st = XGEN_ERR_CUDA;
        cudaSetDevice(prev);
        if (st != XGEN_OK) {
            cudaGetLastError();
            xgen_blockgemm_free(h);
            return st;
        }
    }
    *out = h;
    return XGEN_OK;
}

xgen_status xgen_blockgemm_run(const xgen_blockgemm_packed *hc, const void *x, int64_t m, const void *bias,
                               int32_t relu, void *y, void *stream) {
    xgen_blockgemm_packed *h = const_cast<xgen_blockgemm_packed *>(hc);
    if (!h || !x || !y) return XGEN_ERR_INVALID_ARG;
    const Host &H = h->host;
    const size_t eb = H.dtype == XGEN_F32 ? 4 : 2;
    if (((uintptr_t)x % eb) || ((uintptr_t)y % eb) || ((uintptr_t)bias % 4)) return XGEN_ERR_INVALID_ARG;
    if (m < 1 || m * (int64_t)H.k > 2147483647LL || m * (int64_t)H.c_out > 2147483647LL) return XGEN_ERR_SHAPE;
    {
        const uintptr_t xa = (uintptr_t)x, xe = xa + (size_t)m * H.k * eb, ya = (uintptr_t)y, ye = ya + (size_t)m * H.c_out * eb;
        if (xa < ye && ya < xe) return XGEN_ERR_INVALID_ARG;
    }
    if (h->device < 0) return XGEN_ERR_CUDA;
    GParams P{};
    P.x = x; P.y = y; P.bias = static_cast<const float *>(bias);
    P.stream = reinterpret_cast<const uint4 *>(h->d_stream); P.seg_off = h->d_seg;
    P.m = m; P.k = H.k; P.c_out = H.c_out;
    P.warps = H.warps; P.rows_per_block = H.rows_per_block; P.n_rb = H.n_rb; P.ks = H.ks; P.ns = H.ns;
    P.relu = relu ? 1 : 0;
    P.async_x = (((uintptr_t)x % 4) == 0 && (H.dtype == XGEN_F32 || H.k % 2 == 0)) ? 1 : 0;
    P.vec_y = (((uintptr_t)y % 16) == 0 && (H.c_out * eb) % 16 == 0) ? 1 : 0;
    P.cmd_units = H.max_stage_units + 1;
    const int cols = ((H.warps + 3) / 4) * kRowsPerWarp * kPixPerLane;
    P.tmem_cols = cols <= 128 ? 128 : cols <= 256 ? 256 : 512;
    const size_t smem = smem_bytes(H);
    int prev = 0;
    cudaGetDevice(&prev);
    if (prev != h->device && cudaSetDevice(h->device) != cudaSuccess) return XGEN_ERR_CUDA;
    const void *kern = kernel_for(H.dtype, H.ks);
    xgen_status st = XGEN_OK;
    if (!h->attr_set.load()) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit) != cudaSuccess) st = XGEN_ERR_CUDA;
        else h->attr_set.store(true);
    }
    if (st == XGEN_OK) {
        const long long tiles = (m + kTileM - 1) / kTileM;
        const long long blocks = tiles * H.n_rb;
        if (blocks > 2147483647LL) st = XGEN_ERR_SHAPE;
        else {
            void *args[] = {&P};
            if (cudaLaunchKernel(kern, dim3((unsigned)blocks), dim3((unsigned)H.warps * 32), args, smem, (cudaStream_t)stream) != cudaSuccess) st = XGEN_ERR_CUDA;
            else patconv::count_launch();
        }
    }
    if (st != XGEN_OK) cudaGetLastError();
    if (prev != h->device) cudaSetDevice(prev);
    return st;
}

xgen_status xgen_blockgemm_query(const xgen_blockgemm_packed *h, xgen_blockgemm_stats *stats) {
    if (!h || !stats) return XGEN_ERR_INVALID_ARG;
    *stats = h->host.stats;
    return XGEN_OK;
}

xgen_status xgen_blockgemm_view(const xgen_blockgemm_packed *h, xgen_blockgemm_host_view *view) {
    if (!h || !view) return XGEN_ERR_INVALID_ARG;
    view->units = h->host.stream.data();
    view->n_units = (int64_t)(h->host.stream.size() / 4);
    view->seg_off = h->host.seg_off.data();
    return XGEN_OK;
}

void xgen_blockgemm_free(xgen_blockgemm_packed *h) {
    if (!h) return;
    if (h->device >= 0) {
        int prev = 0;
        cudaGetDevice(&prev);
        if (cudaSetDevice(h->device) == cudaSuccess) {
            if (h->d_stream) cudaFree(h->d_stream);
            if (h->d_seg) cudaFree(h->d_seg);
        }
        cudaSetDevice(prev);
    }
    delete h;
}

}  // extern "C"
