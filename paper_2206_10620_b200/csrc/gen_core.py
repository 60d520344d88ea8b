#!/usr/bin/env python3
"""Generate core_gen.inc: the per-pattern inner code of the convolution kernels.

The paper's low-level optimisation (Sec. 2.3, "Load Redundancy Elimination")
generates, for each pattern, code whose data accesses are all statically
known, and calls it dynamically during execution.  This script is that code
generator for sm_100a.  For a pattern table and a stride it emits one inline
PTX block that interprets a warp's command stream from shared memory.

Commands are 32-byte slots {opcode, operand, -, -, w0, w1, w2, w3}:
  opcode p < NP : kernel command.  The operand is the tensor-memory column of
                  the addressed filter's 8 running sums (2x4 output pixels of
                  this thread).  The block for pattern p multiplies the four
                  weights with the 4 taps x 8 pixels of the register-resident
                  activation patch; tap offsets are immediate register names.
  opcode NP     : LOAD.  The operand is the channel inside the staged chunk;
                  the thread's patch (2x4 pixels plus halo) is read from the
                  staged tile into registers.
  opcode NP + 1 : END of the warp's commands for this chunk.

The running sums live in tensor memory because the filter a command addresses
is data: tensor-memory columns can be addressed at run time, registers cannot.
The pattern selects code, so nothing inside a kernel command is indexed or
branches.

The interpreter is software-pipelined over two register sets (A and B), with
every block emitted once per set.  While command i runs from set A:
  * command i+1 is already decoded in set B, and its row of sums is fetched
    from tensor memory (tcgen05.ld) before command i's arithmetic starts;
  * command i+2 is read from shared memory into set A once command i's weights
    are consumed;
  * the block ends with an indirect branch on set B's opcode (brx.idx).
Between two LOADs every kernel command addresses a different filter, so the
row fetched ahead by a kernel command is never one with a write in flight; a
LOAD (and the block's exit) waits for all writes (tcgen05.wait::st) before it
fetches ahead, which covers a filter that ends one channel and starts the
next.  A row fetched ahead for a LOAD or END command is never used.  The stream segment is staged with two valid
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
    """f2: use packed two-wide fp32 FMAs (fma.rn.f32x2); stride 1 only."""
    assert not (f2 and stride != 1)
    masks = table(np_)
    rows, cols = (6, 4) if stride == 1 else (9, 5)
    npatch = rows * cols
    L = ["{"]
    L.append(" .reg .b32 opA, payA, taA, opB, payB, taB, ad;")
    L.append(" .reg .f32 wA<4>, wB<4>, aA<8>, aB<8>, p<%d>;" % npatch)
    if f2:
        L.append(" .reg .b64 q<%d>, acc<4>, wd<4>;" % (rows * 3))
    # Registers written on one path and read on another must be defined on every
    # path into the branch tables, or register allocation degrades badly.
    if f2:
        for i in range(rows * 3):
            L.append(" mov.b64 q%d, 0;" % i)
    else:
        for i in range(npatch):
            L.append(" mov.f32 p%d, 0f00000000;" % i)
    for i in range(8):
        L.append(" mov.f32 aB%d, 0f00000000;" % i)
    L.append(" mov.b32 taB, %4;")
    for S in "AB":
        L.append(" ts%s: .branchtargets %s;" % (
            S, ",".join("K%s%d" % (S, i) for i in range(len(masks))) + ",LOAD%s,END%s" % (S, S)))

    def fetch(S, off):
        return [" ld.shared.v2.b32 {op%s, pay%s}, [%%0+%d];" % (S, S, off),
                " ld.shared.v4.f32 {w%s0,w%s1,w%s2,w%s3}, [%%0+%d];" % (S, S, S, S, off + 16)]

    def accs(S):
        return "{" + ",".join("a%s%d" % (S, i) for i in range(8)) + "}"

    # prologue: commands 0 and 1 decoded, row of command 0 requested
    L += fetch("A", 0) + fetch("B", 32)
    L.append(" add.u32 %0, %0, 64;")
    L.append(" add.u32 taA, %4, payA;")
    L.append(" tcgen05.wait::st.sync.aligned;")
    L.append(" tcgen05.ld.sync.aligned.32x32b.x8.b32 %s, [taA];" % accs("A"))
    L.append(" brx.idx opA, tsA;")

    for S, O in (("A", "B"), ("B", "A")):
        def prefetch_next(fence):
            r = [" tcgen05.wait::ld.sync.aligned;",             # my own row has arrived
                 " add.u32 ta%s, %%4, pay%s;" % (O, O)]
            if fence:
                r.append(" tcgen05.wait::st.sync.aligned;")     # no write to any row is in flight
            r.append(" tcgen05.ld.sync.aligned.32x32b.x8.b32 %s, [ta%s];" % (accs(O), O))
            return r

        def refill_and_go():
            return fetch(S, 0) + [" add.u32 %0, %0, 32;", " brx.idx op%s, ts%s;" % (O, O)]

        for pi, m in enumerate(masks):
            L.append(" K%s%d:" % (S, pi))
            L += prefetch_next(False)
            taps = [t for t in range(9) if (m >> t) & 1]
            if f2:
                for k in range(4):
                    L.append(" mov.b64 wd%d, {w%s%d, w%s%d};" % (k, S, k, S, k))
                for py in range(4):
                    L.append(" mov.b64 acc%d, {a%s%d, a%s%d};" % (py, S, 2 * py, S, 2 * py + 1))
                for k, t in enumerate(taps):
                    dy, dx = divmod(t, 3)
                    for py in range(4):
                        L.append(" fma.rn.f32x2 acc%d, wd%d, q%d, acc%d;" % (py, k, (py + dy) * 3 + dx, py))
                for py in range(4):
                    L.append(" mov.b64 {a%s%d, a%s%d}, acc%d;" % (S, 2 * py, S, 2 * py + 1, py))
            else:
                for k, t in enumerate(taps):
                    dy, dx = divmod(t, 3)
                    for py in range(4):
                        for px in range(2):
                            pr = (py * stride + dy) * cols + px * stride + dx
                            a = py * 2 + px
                            L.append(" fma.rn.f32 a%s%d, w%s%d, p%d, a%s%d;" % (S, a, S, k, pr, S, a))
            L.append(" tcgen05.st.sync.aligned.32x32b.x8.b32 [ta%s], %s;" % (S, accs(S)))
            L += refill_and_go()

        L.append(" LOAD%s:" % S)
        L += prefetch_next(True)
        L.append(" mad.lo.u32 ad, pay%s, %%2, %%1;" % S)
        for r in range(rows):
            if stride == 1:
                if f2:
                    L.append(" ld.shared.v2.f32 {p0,p1}, [ad];")
                    L.append(" ld.shared.v2.f32 {p2,p3}, [ad+8];")
                    L.append(" mov.b64 q%d, {p0,p1};" % (r * 3))
                    L.append(" mov.b64 q%d, {p1,p2};" % (r * 3 + 1))
                    L.append(" mov.b64 q%d, {p2,p3};" % (r * 3 + 2))
                else:
                    L.append(" ld.shared.v2.f32 {p%d,p%d}, [ad];" % (r * 4, r * 4 + 1))
                    L.append(" ld.shared.v2.f32 {p%d,p%d}, [ad+8];" % (r * 4 + 2, r * 4 + 3))
            else:
                L.append(" ld.shared.v4.f32 {p%d,p%d,p%d,p%d}, [ad];" % tuple(r * 5 + i for i in range(4)))
                L.append(" ld.shared.f32 p%d, [ad+16];" % (r * 5 + 4))
            if r < rows - 1:
                L.append(" add.u32 ad, ad, %3;")
        L += refill_and_go()

        L.append(" END%s:" % S)
        L.append(" bra.uni DONE;")
    L.append(" DONE:")
    L.append(" tcgen05.wait::ld.sync.aligned;")
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
