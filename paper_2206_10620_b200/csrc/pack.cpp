// Host-side packer: pattern masking, filter reorder, kernel reorder and the
// compact command-stream layout (paper Sec. 2.3, "Filter Kernel Reorder and
// Compact FKW Storage").  Pure C++, no CUDA.
//
// Layout idea.  A warp owns one *filter group* (J consecutive output channels) for a
// tile of output pixels; each thread keeps J x T running sums in tensor memory (T = 16
// output pixels per thread at stride 1, 8 at stride 2).  For every
// input channel the group is connected to, the warp loads the activation patch
// of its pixels once into registers (a LOAD command) and then executes one
// *kernel command* per surviving kernel of that channel: the command names the
// filter slot (an address) and the pattern (the code to run), and carries the
// four kept weights.  One small word pair per kernel replaces CSR's index per
// weight, and because the pattern selects straight-line code with fixed
// register operands there is no per-tap index and no branch inside a kernel.
#include <algorithm>
#include <array>
#include <cmath>
#include <cstring>
#include <numeric>

#include "patconv_internal.h"

namespace patconv {

static int popcount9(unsigned m) {
    int n = 0;
    for (int t = 0; t < 9; ++t) n += (m >> t) & 1;
    return n;
}

uint16_t compiled_mask(int np, int idx) {
    if (np <= kNumLibraryMasks) return kLibraryMasks[idx];
    int k = 0;
    for (unsigned m = 0; m < 512; ++m)
        if (popcount9(m) == 4) {
            if (k == idx) return (uint16_t)m;
            ++k;
        }
    return 0;
}

static float half_bits_to_float(uint16_t h) {
    uint32_t sign = (uint32_t)(h & 0x8000u) << 16;
    uint32_t exp = (h >> 10) & 0x1Fu;
    uint32_t man = h & 0x3FFu;
    uint32_t bits;
    if (exp == 0) {
        if (man == 0) {
            bits = sign;
        } else {  // subnormal: normalise
            int e = -1;
            do { man <<= 1; ++e; } while (!(man & 0x400u));
            bits = sign | ((uint32_t)(127 - 15 - e) << 23) | ((man & 0x3FFu) << 13);
        }
    } else if (exp == 31) {
        bits = sign | 0x7F800000u | (man << 13);
    } else {
        bits = sign | ((exp + 127 - 15) << 23) | (man << 13);
    }
    float f;
    std::memcpy(&f, &bits, 4);
    return f;
}

PackConfig choose_pack_config(int c_in, int c_out, xgen_dtype dtype, int stride, bool int_totals) {
    PackConfig c;
    c.channels_per_chunk = c_in <= 4 ? 4 : 8;
    // A warp's running sums take J x (pixels per thread) tensor-memory columns, and an SM
    // has 4 x 512 of them: 128 columns per warp lets 16 warps share an SM.  Integer layers
    // whose exact fp32 partial sums could leave the 24-bit range keep a second row per
    // filter (int32 totals), so they group half as many.
    (void)dtype;
    c.filters_per_group = 128 / pix_per_thread(stride);
    if (int_totals && stride == 2) c.filters_per_group /= 2;
    // Stride 2 groups 16 filters per warp; a layer with fewer than 16 such groups would leave
    // warp slots of its thread block empty, so it groups 8 and runs twice as many warps.
    if (stride == 2 && !int_totals && (c_out + 15) / 16 < 16) c.filters_per_group = 8;
    int groups = (c_out + c.filters_per_group - 1) / c.filters_per_group;
    c.groups_per_block = std::min(groups, int_totals && stride == 1 ? 8 : 16);
    return c;
}

xgen_status parse_layer(const xgen_patconv_desc &d, const void *dense_w, const int16_t *pid_in, PackedHost &out) {
    const int16_t *pid = pid_in;
    if (!dense_w || !pid || !d.pattern_masks) return XGEN_ERR_INVALID_ARG;
    if (d.c_in < 1 || d.c_out < 1) return XGEN_ERR_INVALID_ARG;
    if (d.pad != 1 || (d.stride != 1 && d.stride != 2)) return XGEN_ERR_UNSUPPORTED;
    if (d.dtype != XGEN_F32 && d.dtype != XGEN_F16_F32ACC && d.dtype != XGEN_I8_I32)
        return XGEN_ERR_UNSUPPORTED;
    if (d.num_patterns < 1 || d.num_patterns > kNumAllMasks) return XGEN_ERR_BAD_PATTERN;
    if ((int64_t)d.c_in * d.c_out > (int64_t)1 << 28) return XGEN_ERR_SHAPE;

    const int P = d.num_patterns, cin = d.c_in, cout = d.c_out;
    // --- a1: validate the library and the ids ---------------------------------
    std::vector<int> lib_index(P, -1);  // position in the built-in library, if any
    for (int p = 0; p < P; ++p) {
        unsigned m = d.pattern_masks[p];
        if (m >= 512u || popcount9(m) != 4) return XGEN_ERR_BAD_PATTERN;
        for (int q = 0; q < kNumLibraryMasks; ++q)
            if (kLibraryMasks[q] == m) lib_index[p] = q;
    }
    int max_lib = -1;
    bool all_in_lib = true;
    int64_t k_surv = 0;
    for (int64_t k = 0; k < (int64_t)cin * cout; ++k) {
        int p = pid[k];
        if (p < -1 || p >= P) return XGEN_ERR_BAD_PATTERN;
        if (p < 0) continue;
        if (lib_index[p] < 0) all_in_lib = false;
        max_lib = std::max(max_lib, lib_index[p]);
        ++k_surv;
    }
    const int np = !all_in_lib ? kNumAllMasks : (max_lib < 4 ? 4 : (max_lib < 8 ? 8 : 12));
    // caller pattern id -> index in the compiled table
    std::vector<int> to_compiled(P, 0);
    out = PackedHost();
    out.masks.resize(np);
    for (int q = 0; q < np; ++q) out.masks[q] = compiled_mask(np, q);
    for (int p = 0; p < P; ++p) {
        if (np <= kNumLibraryMasks) {
            to_compiled[p] = lib_index[p] >= 0 && lib_index[p] < np ? lib_index[p] : 0;
        } else {
            for (int q = 0; q < np; ++q)
                if (out.masks[q] == d.pattern_masks[p]) to_compiled[p] = q;
        }
    }

    // Keep the survivors (compiled pattern id and the four kept weights, widened
    // to fp32 exactly) so the layout can be rebuilt for another grouping later.
    out.c_in = cin; out.c_out = cout; out.stride = d.stride; out.dtype = d.dtype; out.np = np;
    out.kpat.assign((size_t)cin * cout, -1);
    out.kw4.assign((size_t)cin * cout * 4, 0u);
    for (int64_t k = 0; k < (int64_t)cin * cout; ++k) {
        int p = pid[k];
        if (p < 0) continue;
        const int q = to_compiled[p];
        out.kpat[k] = (int16_t)q;
        unsigned m = out.masks[q];
        int n = 0;
        for (int t = 0; t < 9; ++t) {
            if (!((m >> t) & 1)) continue;
            float f;
            if (d.dtype == XGEN_F32) f = ((const float *)dense_w)[k * 9 + t];
            else if (d.dtype == XGEN_F16_F32ACC) f = half_bits_to_float(((const uint16_t *)dense_w)[k * 9 + t]);
            else f = (float)((const int8_t *)dense_w)[k * 9 + t];
            std::memcpy(&out.kw4[k * 4 + n++], &f, 4);
        }
    }
    out.stats.kernels_total = (int64_t)cin * cout;
    out.stats.kernels_surviving = k_surv;
    // Integer layers run on exact fp32 FMAs: a sum of u8 x s8 products is exact while its
    // magnitude stays below 2^24, and no partial sum of a filter can exceed 255 x (sum of the
    // magnitudes of its kept weights).  Only if some filter can exceed that are int32 totals
    // kept beside the fp32 sums (and the fp32 sums folded into them in time).
    out.int_totals = false;
    if (d.dtype == XGEN_I8_I32) {
        for (int oc = 0; oc < cout && !out.int_totals; ++oc) {
            double sum_abs = 0.0;
            for (int ic = 0; ic < cin; ++ic) {
                if (out.kpat[(size_t)oc * cin + ic] < 0) continue;
                for (int k = 0; k < 4; ++k) {
                    float f;
                    std::memcpy(&f, &out.kw4[((size_t)oc * cin + ic) * 4 + k], 4);
                    sum_abs += std::fabs((double)f);
                }
            }
            if (255.0 * sum_abs >= 16777216.0) out.int_totals = true;
        }
    }
    return XGEN_OK;
}

xgen_status pack_host(const xgen_patconv_desc &d, const void *dense_w, const int16_t *pid_in,
                      const PackConfig &cfg, PackedHost &out) {
    const xgen_status st = parse_layer(d, dense_w, pid_in, out);
    return st == XGEN_OK ? build_layout(out, cfg) : st;
}

xgen_status build_layout(PackedHost &out, const PackConfig &cfg) {
    const int cin = out.c_in, cout = out.c_out, np = out.np;
    const int16_t *pid = out.kpat.data();           // compiled pattern ids from here on
    const int64_t k_surv = out.stats.kernels_surviving;
    const int J = cfg.filters_per_group, cc = cfg.channels_per_chunk;
    const int wpc = cfg.groups_per_block;
    if (J < 1 || wpc < 1 || cc < 1 || (cc & (cc - 1))) return XGEN_ERR_INVALID_ARG;
    const int n_blocks = ((cout + J - 1) / J + wpc - 1) / wpc;
    const int n_groups = n_blocks * wpc;
    const int n_chunks = (cin + cc - 1) / cc;

    if (cfg.block_rows != 4 && !(cfg.block_rows == 2 && out.stride == 1)) return XGEN_ERR_INVALID_ARG;
    out.J = J; out.wpc = wpc; out.cc = cc;
    out.bh = cfg.block_rows;
    out.tpix = (out.stride == 1 ? 4 : 2) * cfg.block_rows;
    out.slots.clear(); out.max_seg_slots = 0;
    out.n_blocks = n_blocks; out.n_chunks = n_chunks;
    out.slot_oc.assign((size_t)n_groups * J, -1);

    // --- a2: filter reorder.  A filter group is a run of J consecutive output
    // channels (so a thread can store a pixel's J results as one contiguous piece);
    // what is reordered is which groups share a thread block.  Groups are sorted by
    // (surviving kernels desc, pattern histogram, index) and taken wpc at a time: the
    // warps of a block, which share the staged chunks of the input tile (a fast warp can
    // run ahead only by the number of pipeline stages), then carry similar numbers of
    // kernels.
    const int n_runs = (cout + J - 1) / J;
    std::vector<int> cnt(n_runs, 0);
    std::vector<std::vector<int>> hist(n_runs, std::vector<int>(np, 0));
    for (int oc = 0; oc < cout; ++oc)
        for (int ic = 0; ic < cin; ++ic) {
            int p = pid[(size_t)oc * cin + ic];
            if (p >= 0) { ++cnt[oc / J]; ++hist[oc / J][p]; }
        }
    std::vector<int> order(n_runs);
    std::iota(order.begin(), order.end(), 0);
    std::sort(order.begin(), order.end(), [&](int a, int c) {
        if (cnt[a] != cnt[c]) return cnt[a] > cnt[c];
        if (hist[a] != hist[c]) return hist[a] > hist[c];
        return a < c;
    });
    std::vector<int64_t> group_kernels(n_groups, 0);
    for (int i = 0; i < n_runs; ++i) {
        const int g = i;                                   // block i / wpc, warp i % wpc
        for (int j = 0; j < J; ++j) {
            const int oc = order[i] * J + j;
            out.slot_oc[(size_t)g * J + j] = oc < cout ? oc : -1;
        }
        group_kernels[g] = cnt[order[i]];
    }

    // --- a3: kernel reorder + compact store.  Per group and channel: one LOAD,
    // then the group's surviving kernels of that channel ordered by (pattern,
    // slot) so equal patterns (equal code) run back to back.
    out.seg_off.assign((size_t)n_blocks * n_chunks * (wpc + 1), 0);
    out.slots.reserve(((size_t)k_surv + (size_t)n_groups * (cin + n_chunks)) * kSlotWords + 64);
    int64_t n_loads = 0;
    struct Ent { int p, j; };
    std::vector<Ent> ents;
    auto push_slot = [&](uint32_t op, uint32_t operand, const uint32_t *w4) {
        uint32_t s[kSlotWords] = {op, operand, 0, 0, 0, 0, 0, 0};
        if (w4) for (int i = 0; i < 4; ++i) s[4 + i] = w4[i];
        out.slots.insert(out.slots.end(), s, s + kSlotWords);
    };
    for (int b = 0; b < n_blocks; ++b) {
        for (int c = 0; c < n_chunks; ++c) {
            int32_t *so = &out.seg_off[((size_t)b * n_chunks + c) * (wpc + 1)];
            for (int g = 0; g < wpc; ++g) {
                so[g] = (int32_t)(out.slots.size() / kSlotWords);
                const int32_t *soc = &out.slot_oc[((size_t)(b * wpc + g)) * J];
                for (int icl = 0; icl < cc; ++icl) {
                    int ic = c * cc + icl;
                    if (ic >= cin) break;
                    ents.clear();
                    for (int j = 0; j < J; ++j) {
                        if (soc[j] < 0) continue;
                        int p = pid[(size_t)soc[j] * cin + ic];
                        if (p >= 0) ents.push_back({p, j});
                    }
                    if (ents.empty()) continue;  // group not connected to this channel
                    std::sort(ents.begin(), ents.end(), [](const Ent &a, const Ent &e) {
                        return a.p != e.p ? a.p < e.p : a.j < e.j;
                    });
                    push_slot((uint32_t)np, (uint32_t)icl, nullptr);
                    ++n_loads;
                    for (const Ent &e : ents) {
                        const uint32_t *w4 = &out.kw4[((size_t)soc[e.j] * cin + ic) * 4];
                        push_slot((uint32_t)e.p, (uint32_t)(e.j * out.tpix), w4);
                    }
                }
                push_slot((uint32_t)np + 1, 0, nullptr);
            }
            so[wpc] = (int32_t)(out.slots.size() / kSlotWords);
            out.max_seg_slots = std::max(out.max_seg_slots, so[wpc] - so[0]);
            if (out.slots.size() / kSlotWords > (size_t)0x03FFFFFF) return XGEN_ERR_SHAPE;
        }
    }
    const int64_t n_slots = (int64_t)(out.slots.size() / kSlotWords);

    xgen_patconv_stats &s = out.stats;
    s.macs_per_pixel = 4 * k_surv;
    const int wbytes = out.dtype == XGEN_F32 ? 4 : (out.dtype == XGEN_F16_F32ACC ? 2 : 1);
    s.weight_bytes = 4 * k_surv * wbytes;
    const int64_t table_bytes = (int64_t)out.seg_off.size() * 4 + (int64_t)out.slot_oc.size() * 4;
    s.compact_index_bytes = n_slots * 2 + table_bytes;
    s.index_bytes = n_slots * kDevSlotBytes + table_bytes - s.weight_bytes;
    s.csr_index_bytes = 4 * k_surv * 4 + (int64_t)(cout + 1) * 4;
    s.stream_bytes = n_slots * kDevSlotBytes;
    s.filters_per_group = J; s.groups_per_block = wpc; s.n_blocks = n_blocks;
    s.channels_per_chunk = cc; s.n_chunks = n_chunks; s.patterns_compiled = np;
    s.max_segment_slots = out.max_seg_slots;
    s.load_commands = n_loads;
    // Warps of one block wait for each other: what matters is the spread inside a block.
    double worst = 1.0;
    for (int b = 0; b < n_blocks; ++b) {
        int64_t mx = 0, sum = 0, n = 0;
        for (int g = b * wpc; g < (b + 1) * wpc && g < n_runs; ++g) { mx = std::max(mx, group_kernels[g]); sum += group_kernels[g]; ++n; }
        if (sum > 0) worst = std::max(worst, (double)mx * (double)n / (double)sum);
    }
    s.group_imbalance = worst;
    return XGEN_OK;
}

}  // namespace patconv
