"""Generates the PTX text of the tiled kernel's per-chunk dispatch loop (dispatch_s1.inc,
dispatch_s2.inc), which kernels_tiled.cu includes inside one `asm volatile` statement.

Why PTX text: the loop needs a real indexed jump (`brx.idx`) from a warp-uniform byte code to a
straight-line body specialised on (filter slot, pattern); a C++ `switch` is lowered to a compare
tree (about 14 branches per kernel), and accumulator / window registers can only be indexed at
compile time, so each (slot, pattern) pair needs its own body.  Threaded code: every body ends by
fetching the code after next and jumping straight to the next body.

Operands of the asm statement: %0..%31 accumulators acc[g][k] (packed float2, g-major),
%32 code pointer, %33 weight pointer, %34 window pointer (one channel before the chunk),
%35 channel stride, %36 row pitch, %37 offset of the middle window column (all in bytes,
shared-memory addresses as u32).

Byte codes: 0..63 kernel (slot = code >> 3, canonical pattern = code & 7); 64..71 advance
(code - 63) channels and reload the register window; 72 ends the chunk (no other value is ever
dispatched).
"""
import os
import sys

CANON_MASKS = [0x03A, 0x09A, 0x0B8, 0x0B2, 0x01B, 0x036, 0x0D8, 0x1B0]
GROUP = 8
CHUNK = 8
NACC = GROUP * 4


def taps(mask):
    return [t for t in range(9) if mask >> t & 1]


def gen(stride):
    rows = 6 if stride == 1 else 9
    out = []
    emit = out.append
    emit("{")
    emit(".reg .b64 win<%d>;" % (rows * 3))
    emit(".reg .b64 w0, w1, w2, w3;")
    emit(".reg .u32 code, nxt, cp, wp, xp, ra;")
    labels = ["K%d" % c for c in range(GROUP * 8)] + ["ADV%d" % a for a in range(1, CHUNK + 1)] + ["END"]
    emit("TS: .branchtargets " + ", ".join(labels) + ";")
    emit("mov.u32 cp, %%%d;" % NACC)
    emit("mov.u32 wp, %%%d;" % (NACC + 1))
    emit("mov.u32 xp, %%%d;" % (NACC + 2))
    emit("ld.shared.v2.b64 {w0, w1}, [wp];")
    emit("ld.shared.v2.b64 {w2, w3}, [wp+16];")
    emit("add.u32 wp, wp, 32;")
    emit("ld.shared.u8 code, [cp];")
    emit("ld.shared.u8 nxt, [cp+1];")
    emit("add.u32 cp, cp, 2;")
    emit("brx.idx.uni code, TS;")

    def head():  # the code to dispatch next is known a whole body ahead of its jump
        emit("mov.u32 code, nxt;")
        emit("ld.shared.u8 nxt, [cp];")
        emit("add.u32 cp, cp, 1;")

    def tail():
        emit("brx.idx.uni code, TS;")

    for g in range(GROUP):
        for p, mask in enumerate(CANON_MASKS):
            emit("K%d:" % (g * 8 + p))
            head()
            tp = taps(mask)
            for s, t in enumerate(tp):
                u, v = divmod(t, 3)
                for k in range(4):
                    acc = g * 4 + k
                    emit("fma.rn.f32x2 %%%d, win%d, w%d, %%%d;" % (acc, (stride * k + u) * 3 + v, s, acc))
                if s == 1:
                    emit("ld.shared.v2.b64 {w0, w1}, [wp];")
                if s == 3:
                    emit("ld.shared.v2.b64 {w2, w3}, [wp+16];")
            emit("add.u32 wp, wp, 32;")
            tail()
    for a in range(1, CHUNK + 1):
        emit("ADV%d:" % a)
        emit("mad.lo.u32 xp, %%%d, %d, xp;" % (NACC + 3, a))
        if a != CHUNK:
            emit("bra.uni WLOAD;")
    emit("WLOAD:")
    head()
    emit("mov.u32 ra, xp;")
    for r in range(rows):
        emit("ld.shared.b64 win%d, [ra];" % (r * 3))
        if stride == 1:
            emit("ld.shared.b64 win%d, [ra+8];" % (r * 3 + 1))
            emit("ld.shared.b64 win%d, [ra+16];" % (r * 3 + 2))
        else:
            emit("ld.shared.b64 win%d, [ra+8];" % (r * 3 + 2))
        if r != rows - 1:
            emit("add.u32 ra, ra, %%%d;" % (NACC + 4))
    if stride == 2:  # middle column sits at a run-time offset (the even-column plane)
        emit("add.u32 ra, xp, %%%d;" % (NACC + 5))
        for r in range(rows):
            emit("ld.shared.b64 win%d, [ra];" % (r * 3 + 1))
            if r != rows - 1:
                emit("add.u32 ra, ra, %%%d;" % (NACC + 4))
    tail()
    emit("END:")
    emit("}")
    return out


def write(path, lines):
    text = "".join('"%s\\n\\t"\n' % l for l in lines)
    if os.path.exists(path) and open(path).read() == text:
        return
    with open(path, "w") as f:
        f.write(text)


def main(outdir):
    write(os.path.join(outdir, "dispatch_s1.inc"), gen(1))
    write(os.path.join(outdir, "dispatch_s2.inc"), gen(2))


if __name__ == "__main__":
    main(sys.argv[1] if len(sys.argv) > 1 else os.path.dirname(os.path.abspath(__file__)))
