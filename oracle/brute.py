"""Scalar, loop-per-element restatement of the scale search for TINY inputs.

TEST INFRASTRUCTURE ONLY (same standing as tlq_oracle.py; shares nothing with the CUDA path).
Pure Python loops over Python floats, with binary32 roundings made explicit through `struct`, so
that an indexing, broadcasting or transposition mistake in the vectorised oracle shows up as a
disagreement.  It also holds the exhaustive nearest-level search used to pin the rounding rule:
for a fixed step and zero-point the round-to-nearest code of Sec. 2.2 must be the integer level
closest to the value among ALL levels of the n-bit range.
"""
from __future__ import annotations

import math
import struct


def f32(x: float) -> float:
    """Round a Python float (binary64) to binary32, nearest-even."""
    return struct.unpack("<f", struct.pack("<f", x))[0]


def bf16_value(bits: int) -> float:
    return struct.unpack("<f", struct.pack("<I", (int(bits) & 0xFFFF) << 16))[0]


def round_half_even(x: float) -> int:
    f = math.floor(x)
    d = x - f
    if d > 0.5 or (d == 0.5 and f % 2 != 0):
        return int(f) + 1
    return int(f)


def to_bf16(x: float) -> float:
    """Nearest bfloat16 of a positive finite double, ties to even, by exact integer arithmetic."""
    if x == 0.0:
        return 0.0
    m, e = math.frexp(x)            # x = m * 2^e, 0.5 <= m < 1
    q = round_half_even(m * 256.0)  # 8 significand bits
    return math.ldexp(q, e - 8)


def nearest_level(p: float, step: float, zero: int, qmax: int) -> list[int]:
    """All codes q in [0, qmax] minimising |p - (q - zero) * step| (exhaustive)."""
    best, arg = None, []
    for q in range(qmax + 1):
        d = abs(p - (q - zero) * step)
        if best is None or d < best:
            best, arg = d, [q]
        elif d == best:
            arg.append(q)
    return arg


def search(x_bits, w_bits, w_imp, group: int, n_grid: int, bits: int = 4, mode: str = "w4a16", x_fp_bits=None):
    """Exhaustive scale search on nested lists; returns (best index, losses list, per-token table).
    `x_fp_bits`: the full-precision stream of the two-stream objective (the reference output is computed
    from it, everything on the quantized side from x_bits)."""
    n, c1, c2 = len(x_bits), len(x_bits[0]), len(w_bits)
    x = [[bf16_value(v) for v in row] for row in x_bits]
    x_ref = x if x_fp_bits is None else [[bf16_value(v) for v in row] for row in x_fp_bits]
    w = [[bf16_value(v) for v in row] for row in w_bits]
    stat = [max(sum(abs(x[i][c]) for i in range(n)) / n, 2.0 ** -20) for c in range(c1)]
    y_fp = [[sum(w[o][c] * x_ref[i][c] for c in range(c1)) for o in range(c2)] for i in range(n)]
    qmax = (1 << bits) - 1
    losses, table = [], []
    for k in range(n_grid):
        s = [to_bf16(stat[c] ** (k / n_grid)) for c in range(c1)]
        y_q = [[0.0] * c2 for _ in range(n)]
        if mode == "w4a16":
            w_hat = [[0.0] * c1 for _ in range(c2)]
            for o in range(c2):
                for g0 in range(0, c1, group):
                    p = [f32(w[o][c] * s[c]) for c in range(g0, g0 + group)]
                    rng = max(f32(max(p) - min(p)), f32(1e-5))
                    step = f32(rng / qmax)
                    zero = min(max(-round_half_even(f32(min(p) / step)), 0), qmax)
                    for j, c in enumerate(range(g0, g0 + group)):
                        q = min(max(round_half_even(f32(p[j] / step)) + zero, 0), qmax)
                        w_hat[o][c] = f32(f32((q - zero) * step) * f32(1.0 / s[c]))
            for i in range(n):
                for o in range(c2):
                    y_q[i][o] = sum(w_hat[o][c] * x[i][c] for c in range(c1))
        else:
            # "w<n>a<m>": symmetric, step = max|.| / (2^(bits-1) - 1), integers in [-2^(bits-1), 2^(bits-1)-1]
            wn, an = (int(v) for v in mode[1:].split("a"))
            wpos, apos = (1 << (wn - 1)) - 1, (1 << (an - 1)) - 1
            qw, u = [], []
            for o in range(c2):
                p = [f32(w[o][c] * s[c]) for c in range(c1)]
                uo = f32(max(max(abs(v) for v in p), f32(1e-5)) / float(wpos))
                u.append(uo)
                qw.append([min(max(round_half_even(f32(v / uo)), -wpos - 1), wpos) for v in p])
            for i in range(n):
                xt = [f32(x[i][c] * f32(1.0 / s[c])) for c in range(c1)]
                t = f32(max(max(abs(v) for v in xt), f32(1e-5)) / float(apos))
                qx = [min(max(round_half_even(f32(v / t)), -apos - 1), apos) for v in xt]
                for o in range(c2):
                    y_q[i][o] = t * u[o] * sum(qx[c] * qw[o][c] for c in range(c1))
        e = [sum((y_fp[i][o] - y_q[i][o]) ** 2 for o in range(c2)) for i in range(n)]
        table.append(e)
        losses.append(sum(w_imp[i] * e[i] for i in range(n)) / (c2 * sum(w_imp)))
    best = min(range(n_grid), key=lambda k: (losses[k], k))
    return best, losses, table
