"""Re-derive the numeric columns of the golden fixtures with exact rational arithmetic and `math` only.

Run `python tests/golden/make_golden.py` to check the committed files; it imports neither the
oracle nor the CUDA library.  Values: E4M3 closed form, the two hand-worked quantisation groups,
the logistic-function routing examples and the one-token operator evaluation.
"""
import math
import os
import struct
from fractions import Fraction as F

HERE = os.path.dirname(os.path.abspath(__file__))


def f32(x):  # round a Python float (or Fraction) to IEEE fp32, nearest-even
    return struct.unpack("f", struct.pack("f", float(x)))[0]


def e4m3_values():
    vals = []
    for c in range(0x7F):
        e, m = c >> 3, c & 7
        vals.append(F(m, 8) * F(1, 64) if e == 0 else (1 + F(m, 8)) * F(2) ** (e - 7))
    return vals


def e4m3_rne(x):  # exact round-to-nearest-even of a Fraction, saturating
    s = 0x80 if x < 0 else 0
    a = abs(x)
    vals = e4m3_values()
    if a >= vals[-1]:
        return s | 0x7E
    best = min(range(len(vals)), key=lambda c: (abs(vals[c] - a), c & 1))
    return s | best


def check(cond, msg):
    if not cond:
        raise SystemExit("golden mismatch: " + msg)


def main():
    for line in open(os.path.join(HERE, "e4m3_spot_codes.txt")):
        if line.startswith("#") or not line.strip():
            continue
        code, val = line.split()
        c = int(code, 16)
        v = e4m3_values()[c & 0x7F] * (-1 if c & 0x80 else 1)
        check(float(v) == float(val), line)
    rows = {}
    for line in open(os.path.join(HERE, "quant_worked_groups.txt")):
        if line.startswith("#") or not line.strip():
            continue
        name, key, *vals = line.split()
        rows.setdefault(name, {})[key] = vals
    for name, g in rows.items():
        xs = [float(v) for v in g["x"]]
        scale = f32(F(f32(max(abs(v) for v in xs))) / 448)
        check(scale == f32(float(g["scale"][0])), name + " scale")
        for x, b in zip(xs, g["bytes"]):
            r = f32(F(x) / F(scale))
            code = e4m3_rne(F(r))
            if x == 0 and math.copysign(1, x) < 0:
                code = 0x80
            check(code == int(b, 16), f"{name} x={x} -> {code:#x} != {b}")
    sig = lambda z: 1 / (1 + math.exp(-z))
    check(abs(sig(1.0) - 0.7310585786300049) < 1e-15, "softmax")
    s = [sig(z) for z in (2.0, 0.0, -1.0, 1.0)]
    check(abs(s[2] / (s[2] + s[1]) - 0.34975540905421887) < 1e-15, "sigmoid renorm")
    xs = f32(F(1) / 448)
    gate = 448 * xs
    a = f32(gate / (1 + math.exp(-gate)) * 2 * gate)
    hs = f32(F(a) / 448)
    check(e4m3_rne(F(f32(F(a) / F(hs)))) == 0x7E, "hq code")
    y = 448 * hs
    bits = struct.unpack("I", struct.pack("f", y))[0]
    bf = (bits + 0x7FFF + ((bits >> 16) & 1)) >> 16
    check(bf == 0x3FBB, f"one-token out {bf:#x}")
    print("golden fixtures consistent")


if __name__ == "__main__":
    main()
