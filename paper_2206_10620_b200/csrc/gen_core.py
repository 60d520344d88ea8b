#!/usr/bin/env python3
"""Generate core_gen.inc: the per-pattern inner code of the convolution kernels.

The paper's low-level optimisation (Sec. 2.3, "Load Redundancy Elimination")
generates, for each pattern, code whose data accesses are all statically
known, and calls it dynamically during execution.  This script is that code
generator for sm_100a.  For a pattern table and a stride it emits one inline
PTX block that interprets a warp's command stream from shared memory.

Commands are 32-byte slots {opcode, operand, -, -, w0, w1, w2, w3}:
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

Command decoding is software-pipelined over two register sets (A and B), with
every block emitted once per set: while command i runs from set A, command i+1
is already decoded in set B, command i+2 is read from shared memory into set A
once command i's weights are consumed, and the block ends with an indirect
branch on set B's opcode (brx.idx).  Between two LOADs every kernel command
addresses a different filter; a LOAD and the block's exit wait for all
tensor-memory writes (tcgen05.wait::st), which covers a filter that ends one
channel and starts the next.  The stream segment is staged with two valid
spare slots so the look-ahead never reads undefined data.

Operands of every block, in order:
  %0 "+r" shared-memory address of the warp's first command slot
  %1 "r"  shared-memory address of this thread's patch origin in plane 0
  %2 "r"  bytes per channel plane      %3 "r" bytes per tile row
  %4 "r"  tensor-memory address of this warp's first column (lane field set)
"""
import os
import sys

LIBRARY = [0x01B, 0x036, 0x0D8, 0x1B0, 0x03A, 0x09A, 0x0B2, 0x0B8, 0x017, 0x1D0, 0x059, 0x134]
ALL_MASKS = [m for m in range(512) if bin(m).count("1") == 4]


def table(np_):
    return LIBRARY[:np_] if np_ <= 12 else ALL_MASKS


def gen_block(np_, stride, f2):
    """One interpreter block.  Stride 1: a thread owns 4x4 output pixels (16 running
    sums per filter, patch 6x6); stride 2: 2x4 pixels (8 sums, patch 9x5).
    f2: packed two-wide fp32 FMAs (fma.rn.f32x2), stride 1 only."""
    assert not (f2 and stride != 1)
    masks = table(np_)
    bw, bh = (4, 4) if stride == 1 else (2, 4)
    T = bw * bh
    rows = (bh - 1) * stride + 3
    cols = (bw - 1) * stride + 3
    npatch = rows * cols
    npair = cols - 1
    L = ["{"]
    L.append(" .reg .b32 opA, payA, opB, payB, ta, ad;")
    L.append(" .reg .f32 wA<4>, wB<4>, a<%d>, p<%d>;" % (T, npatch if not f2 else cols))
    if f2:
        L.append(" .reg .b64 q<%d>, acc<%d>, wd<4>;" % (rows * npair, T // 2))
    # Registers written on one path and read on another must be defined on every
    # path into the branch tables, or register allocation degrades badly.
    if f2:
        for i in range(rows * npair):
            L.append(" mov.b64 q%d, 0;" % i)
    else:
        for i in range(npatch):
            L.append(" mov.f32 p%d, 0f00000000;" % i)
    for S in "AB":
        L.append(" ts%s: .branchtargets %s;" % (
            S, ",".join("K%s%d" % (S, i) for i in range(len(masks))) + ",LOAD%s,END%s" % (S, S)))

    def fetch(S, off):
        return [" ld.shared.v2.b32 {op%s, pay%s}, [%%0+%d];" % (S, S, off),
                " ld.shared.v4.f32 {w%s0,w%s1,w%s2,w%s3}, [%%0+%d];" % (S, S, S, S, off + 16)]

    accs = "{" + ",".join("a%d" % i for i in range(T)) + "}"

    # prologue: commands 0 and 1 decoded
    L += fetch("A", 0) + fetch("B", 32)
    L.append(" add.u32 %0, %0, 64;")
    L.append(" brx.idx opA, tsA;")

    for S, O in (("A", "B"), ("B", "A")):
        def refill_and_go():
            return fetch(S, 0) + [" add.u32 %0, %0, 32;", " brx.idx op%s, ts%s;" % (O, O)]

        for pi, m in enumerate(masks):
            L.append(" K%s%d:" % (S, pi))
            L.append(" add.u32 ta, %%4, pay%s;" % S)
            L.append(" tcgen05.ld.sync.aligned.32x32b.x%d.b32 %s, [ta];" % (T, accs))
            taps = [t for t in range(9) if (m >> t) & 1]
            if f2:
                for k in range(4):
                    L.append(" mov.b64 wd%d, {w%s%d, w%s%d};" % (k, S, k, S, k))
            L.append(" tcgen05.wait::ld.sync.aligned;")
            if f2:
                for n in range(T // 2):
                    L.append(" mov.b64 acc%d, {a%d, a%d};" % (n, 2 * n, 2 * n + 1))
                for k, t in enumerate(taps):
                    dy, dx = divmod(t, 3)
                    for py in range(bh):
                        for h in range(bw // 2):
                            L.append(" fma.rn.f32x2 acc%d, wd%d, q%d, acc%d;" % (
                                py * (bw // 2) + h, k, (py + dy) * npair + dx + 2 * h, py * (bw // 2) + h))
                for n in range(T // 2):
                    L.append(" mov.b64 {a%d, a%d}, acc%d;" % (2 * n, 2 * n + 1, n))
            else:
                for k, t in enumerate(taps):
                    dy, dx = divmod(t, 3)
                    for py in range(bh):
                        for px in range(bw):
                            pr = (py * stride + dy) * cols + px * stride + dx
                            a = py * bw + px
                            L.append(" fma.rn.f32 a%d, w%s%d, p%d, a%d;" % (a, S, k, pr, a))
            L.append(" tcgen05.st.sync.aligned.32x32b.x%d.b32 [ta], %s;" % (T, accs))
            L += refill_and_go()

        L.append(" LOAD%s:" % S)
        L.append(" tcgen05.wait::st.sync.aligned;")          # no write to any row is in flight
        L.append(" mad.lo.u32 ad, pay%s, %%2, %%1;" % S)
        for r in range(rows):
            if stride == 1:
                if f2:
                    L.append(" ld.shared.v4.f32 {p0,p1,p2,p3}, [ad];")
                    L.append(" ld.shared.v2.f32 {p4,p5}, [ad+16];")
                    for c in range(npair):
                        L.append(" mov.b64 q%d, {p%d,p%d};" % (r * npair + c, c, c + 1))
                else:
                    L.append(" ld.shared.v4.f32 {p%d,p%d,p%d,p%d}, [ad];" % tuple(r * 6 + i for i in range(4)))
                    L.append(" ld.shared.v2.f32 {p%d,p%d}, [ad+16];" % (r * 6 + 4, r * 6 + 5))
            else:
                L.append(" ld.shared.v4.f32 {p%d,p%d,p%d,p%d}, [ad];" % tuple(r * 5 + i for i in range(4)))
                L.append(" ld.shared.f32 p%d, [ad+16];" % (r * 5 + 4))
            if r < rows - 1:
                L.append(" add.u32 ad, ad, %3;")
        L += refill_and_go()

        L.append(" END%s:" % S)
        L.append(" bra.uni DONE;")
    L.append(" DONE:")
    L.append(" tcgen05.wait::st.sync.aligned;")
    L.append("}")
    return L


def main(out_path):
    parts = ["// Generated by gen_core.py -- do not edit.\n"]
    for stride in (1, 2):
        for np_ in (4, 8, 12, 126):
            for f2 in ((0, 1) if stride == 1 else (0,)):
                lines = gen_block(np_, stride, bool(f2))
                parts.append("#define PATCONV_CORE_S%d_NP%d_F%d(sp, tbase, plane_bytes, pitch_bytes, tmem_base) \\\n"
                             % (stride, np_, 2 if f2 else 1))
                parts.append("  asm volatile( \\\n")
                for s in lines:
                    parts.append('    "%s\\n" \\\n' % s)
                parts.append('    : "+r"(sp) : "r"(tbase), "r"(plane_bytes), "r"(pitch_bytes), "r"(tmem_base) : "memory")\n\n')
    tmp = out_path + ".tmp%d" % os.getpid()
    with open(tmp, "w") as f:
        f.write("".join(parts))
    os.replace(tmp, out_path)


if __name__ == "__main__":
    here = os.path.dirname(os.path.abspath(__file__))
    main(sys.argv[1] if len(sys.argv) > 1 else os.path.join(here, "core_gen.inc"))
