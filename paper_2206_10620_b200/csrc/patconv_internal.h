// Internal declarations shared by the packer (host C++) and the CUDA side.
#pragma once
#include <cstdint>
#include <vector>

#include "patconv.h"

namespace patconv {

constexpr int kSlotWords = 8;   // one command slot of the host image = 32 bytes
constexpr int kDevSlotBytes = 48;   // on the device every weight is stored twice (operand pairs)
// A thread owns a 4x4 block of output pixels at stride 1 and a 2x4 block at stride 2;
// a filter's running sums take that many tensor-memory columns.
constexpr int pix_per_thread(int stride) { return stride == 1 ? 16 : 8; }

// The twelve tap sets of the built-in library (bit 3*dy+dx = tap kept): four 2x2
// blocks holding the centre, four T shapes, four edge-plus-centre.  Layers whose
// masks all lie in the first 4, 8 or 12 run with a table of that size; any other
// layer runs with the universal table of all 126 four-of-nine masks.
constexpr int kNumLibraryMasks = 12;
constexpr uint16_t kLibraryMasks[kNumLibraryMasks] = {
    0x01B, 0x036, 0x0D8, 0x1B0, 0x03A, 0x09A, 0x0B2, 0x0B8, 0x017, 0x1D0, 0x059, 0x134};
constexpr int kNumAllMasks = 126;

// Mask number `idx` of the table with `np` entries (np in {4, 8, 12, 126}).
uint16_t compiled_mask(int np, int idx);

struct PackConfig {
    int filters_per_group;   // J
    int groups_per_block;    // warps per thread block
    int channels_per_chunk;  // input channels staged per pipeline step (power of two)
    int block_rows = 4;      // rows of the pixel block a thread owns: 4, or 2 (stride 1 only: 4x2 pixels)
};

// Host image of a packed layer.
struct PackedHost {
    int c_in = 0, c_out = 0, stride = 1;
    xgen_dtype dtype = XGEN_F32;
    int J = 0, wpc = 0, cc = 0, np = 0;          // np: compiled pattern-table size
    int bh = 4, tpix = 16;                        // block rows and output pixels of a thread (tensor-memory columns per filter)
    int n_blocks = 0, n_chunks = 0;
    int max_seg_slots = 0;
    std::vector<uint32_t> slots;                  // kSlotWords words per command
    std::vector<int32_t> seg_off;                 // [n_blocks * n_chunks * (wpc + 1)]
    std::vector<int32_t> slot_oc;                 // [n_blocks * wpc * J], -1 = empty slot
    std::vector<uint16_t> masks;                  // [np]
    std::vector<int16_t> kpat;                    // [c_out * c_in] compiled pattern id, -1 = removed
    std::vector<uint32_t> kw4;                    // [c_out * c_in * 4] kept weights as fp32 bits
    bool int_totals = false;                      // i8: some filter's exact fp32 sums could leave the 24-bit range
    xgen_patconv_stats stats{};
};

// Default grouping for a layer shape (int_totals: see PackedHost).
PackConfig choose_pack_config(int c_in, int c_out, xgen_dtype dtype, int stride, bool int_totals);

// Validate the description and keep the surviving kernels (pattern ids, kept weights).  No CUDA call.
xgen_status parse_layer(const xgen_patconv_desc &desc, const void *dense_w, const int16_t *pid, PackedHost &out);

// Validate the description and build the host image.  No CUDA call.
xgen_status pack_host(const xgen_patconv_desc &desc, const void *dense_w, const int16_t *pid,
                      const PackConfig &cfg, PackedHost &out);

// Rebuild slots / seg_off / slot_oc / stats of an already parsed layer for a grouping.
xgen_status build_layout(PackedHost &p, const PackConfig &cfg);

// Every kernel launch of the library counts itself here (xgen_patconv_launch_count).
void count_launch();

}  // namespace patconv
