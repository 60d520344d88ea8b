#!/usr/bin/env python3
"""Generate core_gen.inc: the per-pattern inner code of the convolution kernels.

The paper's low-level optimisation (Sec. 2.3, "Load Redundancy Elimination")
generates, for each pattern, code whose data accesses are all statically
known, and calls it dynamically during execution.  This script is that code
generator for sm_100a.  For a pattern table and a stride it emits one inline
PTX block that interprets a warp's command stream from shared memory.

Commands are 48-byte slots {opcode, operand, -, -, w0, w0, w1, w1, w2, w2, w3, w3}
(every kept weight twice, so one 64-bit register pair feeds a two-wide FMA):
  opcode p < NP : kernel command.  The operand is the tensor-memory column of
                  the addressed filter's running sums (one per output pixel of
                  this thread: 4x4 pixels at stride 1, 2x4 at stride 2).  The
                  block for pattern p multiplies the four weights with the 4
                  taps of every pixel, read from the register-resident
                  activation patch; tap offsets are immediate register names.
  opcode NP     : LOAD.  The operand is the channel inside the staged chunk;
                  the thread's patch (its pixels plus halo) is read from the
                  staged tile into registers.
  opcode NP + 1 : END of the warp's commands for this chunk.

The running sums live in tensor memory because the filter a command addresses
is data: tensor-memory columns can be addressed at run time, registers cannot
(a row round trip is about 40 cycles).  The pattern selects code, so nothing
inside a kernel command is indexed or branches.

All arithmetic is fma.rn.f32x2 on pixel pairs two input columns apart: at
stride 1 a thread's row of four pixels splits into the pairs (0,2) and (1,3),
at stride 2 its two pixels form one pair.  A tap at column offset dx then reads
the input pair (dx, dx+2) (or (dx+1, dx+3)), and the staged tile stores exactly
those pairs, so a LOAD is plain 128-bit shared-memory loads straight into the
64-bit operand registers: per tile row and thread, half 0 holds the input
columns (0,2,1,3) and half 1 holds (2,4,3,5) (stride 2: (2,4)).  The two halves
are separate arrays (operands %1 and %5) so that the loads of a quarter warp
fall into distinct banks.

Every block starts by asking tensor memory for its row and shared memory for
its weights and for the opcode and operand of the following command, waits for
the row, runs its FMAs and ends with an indirect branch on that next opcode
(brx.idx): the loads overlap the row fetch, the next opcode is long there when
the branch needs it, and one copy of each block keeps the code small enough to
stay in the instruction cache.  Between two LOADs every kernel command
addresses a different filter; a LOAD and the block's exit wait for all
tensor-memory writes (tcgen05.wait::st), which covers a filter that ends one
channel and starts the next.  The stream segment is staged with valid spare
slots behind it so the look-ahead never reads undefined data.

Operands of every block, in order:
  %0 "+r" shared-memory address of the warp's first command slot
  %1 "r"  shared-memory address of this thread's patch origin, half 0 of plane 0
  %2 "r"  bytes per channel plane      %3 "r" bytes per tile row
  %4 "r"  tensor-memory address of this warp's first column (lane field set)
  %5 "r"  shared-memory address of this thread's patch origin, half 1 of plane 0
"""
import os
import sys

LIBRARY = [0x01B, 0x036, 0x0D8, 0x1B0, 0x03A, 0x09A, 0x0B2, 0x0B8, 0x017, 0x1D0, 0x059, 0x134]
ALL_MASKS = [m for m in range(512) if bin(m).count("1") == 4]
SLOT_BYTES = 48


def table(np_):
    return LIBRARY[:np_] if np_ <= 12 else ALL_MASKS


def gen_block(np_, stride, bh=4):
    """One interpreter block.  Stride 1: a thread owns 4x4 output pixels (16 running
    sums per filter, patch 6 rows x 4 pairs) or, in the small-block form for images
    that would leave most lanes of a 4x4 tiling idle, 4x2 pixels (8 sums, patch 4 rows
    x 4 pairs); stride 2: 2x4 pixels (8 sums, patch 9 rows x 3 pairs)."""
    masks = table(np_)
    bw = 4 if stride == 1 else 2
    T = bw * bh
    rows = (bh - 1) * stride + 3
    ppr = 4 if stride == 1 else 3            # operand pairs per patch row
    L = ["{"]
    L.append(" .reg .b32 op, pay, ta, adA, adB;")
    L.append(" .reg .b32 a<%d>;" % T)
    L.append(" .reg .b64 q<%d>, acc<%d>, wd<4>;" % (rows * ppr, T // 2))
    # Registers written on one path and read on another must be defined on every
    # path into the branch table, or register allocation degrades badly.
    for i in range(rows * ppr):
        L.append(" mov.b64 q%d, 0;" % i)
    L.append(" ts: .branchtargets %s;" % (",".join("K%d" % i for i in range(len(masks))) + ",LOAD,END"))

    accs = "{" + ",".join("a%d" % i for i in range(T)) + "}"

    def next_header():
        # opcode and operand of the following command; %0 moves on to it
        return [" ld.shared.v2.b32 {op, pay}, [%%0+%d];" % SLOT_BYTES,
                " add.u32 %%0, %%0, %d;" % SLOT_BYTES]

    # prologue: command 0 decoded
    L.append(" ld.shared.v2.b32 {op, pay}, [%0];")
    L.append(" brx.idx.uni op, ts;")

    for pi, m in enumerate(masks):
        L.append(" K%d:" % pi)
        L.append(" add.u32 ta, %4, pay;")
        L.append(" tcgen05.ld.sync.aligned.32x32b.x%d.b32 %s, [ta];" % (T, accs))
        L.append(" ld.shared.v2.b64 {wd0, wd1}, [%0+16];")
        L.append(" ld.shared.v2.b64 {wd2, wd3}, [%0+32];")
        L += next_header()
        taps = [t for t in range(9) if (m >> t) & 1]
        L.append(" tcgen05.wait::ld.sync.aligned;")
        for n in range(T // 2):
            L.append(" mov.b64 acc%d, {a%d, a%d};" % (n, 2 * n, 2 * n + 1))
        for k, t in enumerate(taps):
            dy, dx = divmod(t, 3)
            for py in range(bh):
                if stride == 1:
                    for h in range(2):
                        L.append(" fma.rn.f32x2 acc%d, wd%d, q%d, acc%d;" % (
                            py * 2 + h, k, (py + dy) * ppr + dx + h, py * 2 + h))
                else:
                    L.append(" fma.rn.f32x2 acc%d, wd%d, q%d, acc%d;" % (
                        py, k, (2 * py + dy) * ppr + dx, py))
        for n in range(T // 2):
            L.append(" mov.b64 {a%d, a%d}, acc%d;" % (2 * n, 2 * n + 1, n))
        L.append(" tcgen05.st.sync.aligned.32x32b.x%d.b32 [ta], %s;" % (T, accs))
        L.append(" brx.idx.uni op, ts;")

    L.append(" LOAD:")
    L.append(" tcgen05.wait::st.sync.aligned;")          # no write to any row is in flight
    L.append(" mad.lo.u32 adA, pay, %2, %1;")
    L.append(" mad.lo.u32 adB, pay, %2, %5;")
    L += next_header()
    for r in range(rows):
        L.append(" ld.shared.v2.b64 {q%d,q%d}, [adA];" % (r * ppr, r * ppr + 1))
        if stride == 1:
            L.append(" ld.shared.v2.b64 {q%d,q%d}, [adB];" % (r * ppr + 2, r * ppr + 3))
        else:
            L.append(" ld.shared.b64 q%d, [adB];" % (r * ppr + 2))
        if r < rows - 1:
            L.append(" add.u32 adA, adA, %3;")
            L.append(" add.u32 adB, adB, %3;")
    L.append(" brx.idx.uni op, ts;")

    L.append(" END:")
    L.append(" bra.uni DONE;")
    L.append(" DONE:")
    L.append(" tcgen05.wait::st.sync.aligned;")
    L.append("}")
    return L


def main(out_path):
    parts = ["// Generated by gen_core.py -- do not edit.\n"]
    for stride, bh, tag in ((1, 4, "S1"), (2, 4, "S2"), (1, 2, "S1H2")):
        for np_ in (4, 8, 12, 126):
            lines = gen_block(np_, stride, bh)
            parts.append("#define PATCONV_CORE_%s_NP%d(sp, baseA, plane_bytes, pitch_bytes, tmem_base, baseB) \\\n"
                         % (tag, np_))
            parts.append("  asm volatile( \\\n")
            for s in lines:
                parts.append('    "%s\\n" \\\n' % s)
            parts.append('    : "+r"(sp) : "r"(baseA), "r"(plane_bytes), "r"(pitch_bytes), "r"(tmem_base), "r"(baseB) : "memory")\n\n')
    tmp = out_path + ".tmp%d" % os.getpid()
    with open(tmp, "w") as f:
        f.write("".join(parts))
    os.replace(tmp, out_path)


if __name__ == "__main__":
    here = os.path.dirname(os.path.abspath(__file__))
    main(sys.argv[1] if len(sys.argv) > 1 else os.path.join(here, "core_gen.inc"))
