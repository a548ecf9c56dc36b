"""Writes ``generated/tiled_cases.inc``: the inner loop of the tiled kernel as inline PTX, one macro per blocking.

Why PTX text.  The kernels of a (filter block, channel chunk) arrive as a stream of 32-byte records
{w0, w1, w2, w3, descriptor, pad x3}.  Every record is executed by straight-line code specialised for its
(accumulator slot, pattern): 4 taps x TY x 4 pixels of FFMA with compile-time register numbers (the branch-free,
pattern-specialised loops of Sections 5.2/5.4).  The code for the next record is reached with ONE warp-uniform
indirect branch (``brx.idx`` over a ``.branchtargets`` table) issued at the end of the current body -- a threaded
interpreter.  A C++ ``switch`` over the same cases compiles to a tree of compares and branches (measured: more
control instructions than FMAs), and C++ has no computed goto; PTX has.

Macro ``PATDNN_INTERP_<TY>_<FR>_<F32|F16>(ACC, EP, PBASE, PITCHB, PL, PR)`` expands to one ``asm volatile`` with
    %0 .. %(FR*TY*4-1)   ACC[j][y][x]   read-write float accumulators
    EP       shared-space address of the first record of the segment
    PBASE    shared-space address of this lane's patch origin (row 0, column 0 of its tile) in channel 0
    PITCHB   shared-memory row pitch in bytes
    PL, PR   1 if the lane must read its left / right halo column from shared memory (first / last lane of the warp,
             or tile at the image border where the stored zero pad is read), else the halo comes by shuffle
Record codes (descriptor & 1023): slot*NPAT + pattern = FMA body; FR*NPAT = load the patch of the channel whose byte
offset is descriptor >> 10; FR*NPAT + 1 = end of segment.
Body of (j, p): for the i-th kept tap t of builtin pattern p:  ACC[j][y][x] += w_i * patch[y + t/3][x + t%3].
"""
from __future__ import annotations

import os
import sys

BUILTIN_MASKS = (0x01B, 0x036, 0x0D8, 0x1B0, 0x03A, 0x0B8, 0x09A, 0x0B2, 0x017, 0x1D0, 0x059, 0x134)
CONFIGS = ((4, 8), (4, 4), (2, 8))      # (TY, FR)
HERE = os.path.dirname(os.path.abspath(__file__))
OUT = os.path.join(HERE, "generated", "tiled_cases.inc")
RECORD_BYTES = 32


def taps(mask: int):
    return [t for t in range(9) if (mask >> t) & 1]


def emit_config(ty: int, fr: int, half: bool) -> str:
    npat = len(BUILTIN_MASKS)
    n_acc = fr * ty * 4
    rows = ty + 2
    EP, PBASE, PITCHB, PL, PR = (f"%{n_acc + i}" for i in range(5))

    def acc(j, y, x):
        return f"%{(j * ty + y) * 4 + x}"

    def patch(r, c):
        return f"p{r * 6 + c}"

    L = ["{"]
    L.append(f".reg .f32 p<{rows * 6}>;")
    L.append(".reg .f32 w0, w1, w2, w3;")
    L.append(".reg .u32 d, code, ep, a;")
    if half:
        L.append(".reg .b32 h0, h1; .reg .b16 q0, q1, q2, q3, qe;")
    L.append(".reg .pred pl, pr;")
    labels = [f"K{j}_{p}" for j in range(fr) for p in range(npat)] + ["KLOAD", "KEND"]
    L.append("tbl: .branchtargets " + ", ".join(labels) + ";")
    L.append(f"mov.u32 ep, {EP};")
    L.append(f"setp.ne.u32 pl, {PL}, 0;")
    L.append(f"setp.ne.u32 pr, {PR}, 0;")
    L.append("ld.shared.u32 d, [ep+16];")
    L.append("DISP:")
    L.append("and.b32 code, d, 1023;")
    L.append("brx.idx.uni code, tbl;")
    for j in range(fr):
        for p in range(npat):
            L.append(f"K{j}_{p}:")
            L.append("ld.shared.v4.f32 {w0, w1, w2, w3}, [ep];")
            L.append(f"ld.shared.u32 d, [ep+{RECORD_BYTES + 16}];")
            L.append(f"add.u32 ep, ep, {RECORD_BYTES};")
            for i, t in enumerate(taps(BUILTIN_MASKS[p])):          # tap-major: consecutive FMAs are independent
                for y in range(ty):
                    for x in range(4):
                        a = acc(j, y, x)
                        L.append(f"fma.rn.f32 {a}, w{i}, {patch(y + t // 3, x + t % 3)}, {a};")
            L.append("bra.uni DISP;")
    L.append("KLOAD:")
    L.append("shr.u32 a, d, 10;")
    L.append(f"add.u32 a, a, {PBASE};")
    L.append(f"ld.shared.u32 d, [ep+{RECORD_BYTES + 16}];")
    L.append(f"add.u32 ep, ep, {RECORD_BYTES};")
    for r in range(rows):
        m = [patch(r, c) for c in range(6)]
        if half:
            L.append("ld.shared.v2.b32 {h0, h1}, [a];")
            L.append("mov.b32 {q0, q1}, h0;")
            L.append("mov.b32 {q2, q3}, h1;")
            for c in range(4):
                L.append(f"cvt.f32.f16 {m[c + 1]}, q{c};")
        else:
            L.append(f"ld.shared.v4.f32 {{{m[1]}, {m[2]}, {m[3]}, {m[4]}}}, [a];")
        L.append(f"shfl.sync.up.b32 {m[0]}, {m[4]}, 1, 0, 0xffffffff;")
        L.append(f"shfl.sync.down.b32 {m[5]}, {m[1]}, 1, 31, 0xffffffff;")
        if half:
            L.append("@pl ld.shared.b16 qe, [a+-2];")
            L.append(f"@pl cvt.f32.f16 {m[0]}, qe;")
            L.append("@pr ld.shared.b16 qe, [a+8];")
            L.append(f"@pr cvt.f32.f16 {m[5]}, qe;")
        else:
            L.append(f"@pl ld.shared.f32 {m[0]}, [a+-4];")
            L.append(f"@pr ld.shared.f32 {m[5]}, [a+16];")
        if r + 1 < rows:
            L.append(f"add.u32 a, a, {PITCHB};")
    L.append("bra.uni DISP;")
    L.append("KEND:")
    L.append("}")
    text = "".join(f'    "{ln}\\n" \\\n' for ln in L)
    outs = ", ".join(f'"+f"(ACC[{j}][{y}][{x}])' for j in range(fr) for y in range(ty) for x in range(4))
    ins = '"r"(EP), "r"(PBASE), "r"(PITCHB), "r"(PL), "r"(PR)'
    name = f"PATDNN_INTERP_{ty}_{fr}_{'F16' if half else 'F32'}"
    return (f"#define {name}(ACC, EP, PBASE, PITCHB, PL, PR) \\\n    asm volatile( \\\n{text}"
            f"    : {outs} \\\n    : {ins} \\\n    : \"memory\")\n")


def generate(path: str = OUT) -> str:
    body = ("// GENERATED by gen_cases.py -- do not edit.  Threaded interpreter over kernel records: straight-line FMA\n"
            "// bodies per (slot, pattern), one brx.idx per record; see gen_cases.py for operands and record format.\n"
            "#pragma once\n\n")
    body += "\n".join(emit_config(ty, fr, half) for ty, fr in CONFIGS for half in (False, True))
    os.makedirs(os.path.dirname(path), exist_ok=True)
    if not os.path.exists(path) or open(path).read() != body:
        with open(path, "w") as fh:
            fh.write(body)
    return path


if __name__ == "__main__":
    print(generate(sys.argv[1] if len(sys.argv) > 1 else OUT))
