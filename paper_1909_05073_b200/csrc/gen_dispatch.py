"""Generates the PTX text of the tiled kernel's per-chunk dispatch loop (dispatch_s<stride>.inc for
pattern sets inside the canonical eight, dispatch_s<stride>w.inc for any other set,
dispatch_s<stride>t.inc for the canonical sets with 8 instead of 4 output rows per lane), which
kernels_tiled.cu includes inside one `asm volatile` statement.

Why PTX text, and why this shape (all measured on B200):
 * accumulator and window registers can only be named at compile time, so every distinct
   combination that the code must reach needs its own straight-line body;
 * a warp-uniform jump to a *changing* target (`brx.idx`) costs ~100 cycles, which other warps can
   hide only while the bodies being jumped between fit the ~8 KB instruction cache of an SM
   sub-partition; bodies specialised on (filter slot, pattern) are 24-47 KB and ran at 6-16 % of
   the FP32 peak, a C++ `switch` (lowered to a compare tree) no better, predicated-off FFMA2 cost
   as much as executed ones;
 * so the filter slot is taken out of the code: accumulators live in Tensor Memory (TMEM), which is
   addressed at run time.  A body is specialised on the pattern only: it waits for
   the slot's 8 accumulator columns (requested by the previous body), runs the 16 packed FMAs of
   the 4 taps, writes the columns back, requests the next kernel's columns, then jumps.

Shared-memory loads, TMEM loads and TMEM stores all pass through one memory-instruction queue
that retires roughly one instruction per 7-9 cycles per scheduler, whatever its width; with 16
packed FMAs (32 pipe cycles) per kernel that queue is the next limit, so the loop is written to
issue as few such instructions as it can: one 16-byte load for a kernel's four weights (pairs
{w,w} are formed by register moves), one 16-byte load per record of codes (shifted out of four
registers), one TMEM load and one TMEM store of 8 columns, and nine 16-byte loads per
channel window (the staged tile is stored column-major so that two rows come with one load).

Operands of the asm statement (all u32): %0 code pointer (the block's first record), %1 weight
pointer (its first kernel), %2 window pointer (one channel before the chunk), %3 channel stride,
%4 column stride of the staged tile, %5 offset of the middle window column (bytes, shared-memory
addresses), %6 TMEM address of the warp's slot 0, %7 the entry code (an advance code that leads to the block's
first channel).

Two code formats (16-byte records, a run of kernel codes closed by one terminator):
 * narrow (canonical sets): one byte per code, 15 kernels to a record.  Low nibble 0..7 = kernel
   with that canonical pattern, high nibble = filter slot; low nibble 8 = advance (high nibble, may
   be 0) channels, reload the register window and fetch the next record; 9 = end of the block.
   Eight bodies, ~8 KB of hot code: what a scheduler's instruction cache holds.
 * wide (any set of 4-of-9 masks): two bytes per code, 7 kernels to a record.  Low byte = jump
   index, high byte = filter slot or channels to advance.  Index 0 = advance, 1 = end, 2 = fetch
   the next record (the channel has more kernels than a record holds), 3..128 = kernel whose mask
   has that body (`body_masks()`: the canonical eight first, then every other mask with four bits
   in ascending order; the packer enumerates them the same way).  There is a body for each of the
   126 masks (~110 KB of code per stride); a layer touches its own patterns' bodies only.
   Measured: the canonical sets run 6-20 % slower in this format than in the narrow one (fewer
   kernels per record, a larger jump table), which is why both exist.
"""
import os
import sys

CANON_MASKS = [0x03A, 0x09A, 0x0B8, 0x0B2, 0x01B, 0x036, 0x0D8, 0x1B0]


def body_masks():
    """Mask of every body, by jump index (the packer enumerates them the same way)."""
    rest = [m for m in range(512) if bin(m).count("1") == 4 and m not in CANON_MASKS]
    return CANON_MASKS + rest


def taps(mask):
    return [t for t in range(9) if mask >> t & 1]


def gen(stride, wide, R=4):
    """R = output rows per lane and sub-tile: a body runs 4 * R packed FMAs on 2 * R TMEM columns."""
    rows = stride * (R - 1) + 3
    nv = 2 * R                      # TMEM columns (32-bit registers) of one filter slot
    out = []
    emit = out.append
    emit("{")
    emit(".reg .b32 a<%d>;" % nv)
    emit(".reg .b32 s<%d>;" % nv)
    emit(".reg .b64 acc<%d>;" % R)
    emit(".reg .b64 win<%d>;" % (rows * 3))
    emit(".reg .b64 w0, w1, w2, w3;")
    emit(".reg .b32 r0, r1, r2, r3;")          # raw weights of the next kernel
    emit(".reg .b32 c0, c1, c2, c3;")          # the current record of byte codes
    emit(".reg .u32 code, idx, cp, wp, xp, ra, ta, tn, tq;")
    masks = body_masks()
    assert len(masks) == 126
    if wide:
        # the terminators have the lowest indices, then the bodies in body_masks() order
        emit("TS: .branchtargets " + ", ".join(["ADV", "END", "CONT"] + ["P%d" % p for p in range(len(masks))]) + ";")
    else:
        emit("TS: .branchtargets " + ", ".join(["P%d" % p for p in range(8)] + ["ADV", "END"]) + ";")
    emit("mov.u32 cp, %0;")
    emit("mov.u32 wp, %1;")
    emit("mov.u32 xp, %2;")
    emit("mov.u32 tq, %6;")
    emit("mov.u32 code, %7;")
    emit("ld.shared.v4.b32 {r0, r1, r2, r3}, [wp];")
    emit("add.u32 wp, wp, 16;")
    emit("tcgen05.wait::st.sync.aligned;")
    emit("bra.uni ADV;")                      # the entry code leads to the block's first channel

    A8 = "{" + ", ".join("a%d" % i for i in range(nv)) + "}"
    S8 = "{" + ", ".join("s%d" % i for i in range(nv)) + "}"
    slot_shift = 3 if R == 4 else 4

    def prep():
        """Shift the next byte code out of the record registers; decode its jump index and the
        TMEM address of its filter slot."""
        if wide:
            emit("and.b32 code, c0, 65535;")
            emit("shf.r.wrap.b32 c0, c0, c1, 16;")
            emit("shf.r.wrap.b32 c1, c1, c2, 16;")
            emit("shf.r.wrap.b32 c2, c2, c3, 16;")
            emit("shr.u32 c3, c3, 16;")
            emit("and.b32 idx, code, 255;")
            emit("shr.u32 tn, code, 8;")
        else:
            emit("and.b32 code, c0, 255;")
            emit("shf.r.wrap.b32 c0, c0, c1, 8;")
            emit("shf.r.wrap.b32 c1, c1, c2, 8;")
            emit("shf.r.wrap.b32 c2, c2, c3, 8;")
            emit("shr.u32 c3, c3, 8;")
            emit("and.b32 idx, code, 15;")
            emit("shr.u32 tn, code, 4;")
        emit("shl.b32 tn, tn, %d;" % slot_shift)
        emit("add.u32 tn, tn, tq;")

    def jump():
        emit("mov.u32 ta, tn;")
        emit("brx.idx.uni idx, TS;")

    # Kernel bodies.  On entry: the slot's 8 accumulator columns were requested by the previous
    # body (`a`), the kernel's raw weights are in r0..r3.  The body forms the {w,w} pairs, requests
    # the next kernel's weights, runs the 16 FMAs, stores the columns and only then requests the
    # next slot's columns (inside a channel every kernel has a different slot, so that load never
    # follows a store to the same columns; stores are drained where the channel changes).
    def body(p, mask):
        tp = taps(mask)
        emit("P%d:" % p)
        emit("mov.b64 w0, {r0, r0};")
        emit("mov.b64 w1, {r1, r1};")
        emit("mov.b64 w2, {r2, r2};")
        emit("mov.b64 w3, {r3, r3};")
        emit("ld.shared.v4.b32 {r0, r1, r2, r3}, [wp];")
        emit("add.u32 wp, wp, 16;")
        prep()
        emit("tcgen05.wait::ld.sync.aligned;")
        for k in range(R):
            emit("mov.b64 acc%d, {a%d, a%d};" % (k, 2 * k, 2 * k + 1))
        for s_, t in enumerate(tp):
            u, v = divmod(t, 3)
            for k in range(R):
                emit("fma.rn.f32x2 acc%d, win%d, w%d, acc%d;" % (k, (stride * k + u) * 3 + v, s_, k))
        for k in range(R):
            emit("mov.b64 {s%d, s%d}, acc%d;" % (2 * k, 2 * k + 1, k))
        emit("tcgen05.st.sync.aligned.32x32b.x%d.b32 [ta], %s;" % (nv, S8))
        emit("tcgen05.ld.sync.aligned.32x32b.x%d.b32 %s, [tn];" % (nv, A8))
        jump()

    for p in range(len(CANON_MASKS)):
        body(p, masks[p])

    # Advance: `code` >> 8 channels further, reload the window (column-major tile: two rows per
    # 16-byte load) and fetch the next record of codes.
    emit("ADV:")
    emit("tcgen05.wait::ld.sync.aligned;")  # the speculative load issued before this jump
    emit("tcgen05.wait::st.sync.aligned;")  # a slot may come back in the next channel
    emit("shr.u32 ra, code, %d;" % (8 if wide else 4))
    emit("mad.lo.u32 xp, ra, %3, xp;")
    emit("ld.shared.v4.b32 {c0, c1, c2, c3}, [cp];")
    emit("add.u32 cp, cp, 16;")
    cols = [("xp", 0), ("xp", 1), ("xp", 2)]
    for v in range(3):
        if stride == 1:
            emit("mad.lo.u32 ra, %%4, %d, xp;" % v) if v else emit("mov.u32 ra, xp;")
        else:
            # staged columns: odd plane first; the middle (even) column sits at a run-time offset
            if v == 0:
                emit("mov.u32 ra, xp;")
            elif v == 1:
                emit("add.u32 ra, xp, %5;")
            else:
                emit("add.u32 ra, xp, %4;")
        for r in range(0, rows - 1, 2):
            emit("ld.shared.v2.b64 {win%d, win%d}, [ra+%d];" % (r * 3 + v, (r + 1) * 3 + v, r * 8))
        if rows % 2:
            emit("ld.shared.b64 win%d, [ra+%d];" % ((rows - 1) * 3 + v, (rows - 1) * 8))
    prep()
    emit("tcgen05.ld.sync.aligned.32x32b.x%d.b32 %s, [tn];" % (nv, A8))
    jump()
    if wide:
        # Continue: the channel has more kernels than a record holds; fetch the next record.
        emit("CONT:")
        emit("tcgen05.wait::ld.sync.aligned;")  # the speculative load issued before this jump
        emit("ld.shared.v4.b32 {c0, c1, c2, c3}, [cp];")
        emit("add.u32 cp, cp, 16;")
        prep()
        emit("tcgen05.ld.sync.aligned.32x32b.x%d.b32 %s, [tn];" % (nv, A8))
        jump()
    emit("END:")
    emit("tcgen05.wait::ld.sync.aligned;")
    emit("tcgen05.wait::st.sync.aligned;")
    if wide:
        emit("bra.uni DONE;")
        # bodies of the other 118 masks, behind the hot region of the canonical sets
        for p in range(len(CANON_MASKS), len(masks)):
            body(p, masks[p])
    emit("DONE:")
    emit("}")
    return out


def write(path, lines):
    text = "".join('"%s\\n\\t"\n' % l for l in lines)
    if os.path.exists(path) and open(path).read() == text:
        return
    with open(path, "w") as f:
        f.write(text)


def main(outdir):
    for stride in (1, 2):
        write(os.path.join(outdir, "dispatch_s%d.inc" % stride), gen(stride, False))
        write(os.path.join(outdir, "dispatch_s%dw.inc" % stride), gen(stride, True))
        write(os.path.join(outdir, "dispatch_s%dt.inc" % stride), gen(stride, False, 8))


if __name__ == "__main__":
    main(sys.argv[1] if len(sys.argv) > 1 else os.path.dirname(os.path.abspath(__file__)))
