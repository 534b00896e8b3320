"""Writes tests/golden/decision_thresholds.txt: the float32 bit patterns of the thresholds that the decision
stage compares against (Eq. 9: p >= tau as logp >= ln tau; the clip bounds of Eq. 7 / Eq. 10 as
ln(1 + eps_high), ln(1 - eps_low)).

Independent of the oracle and of the CUDA library: the logarithm is evaluated with Python's `decimal`
module at 60 significant digits on the exact value of the float32 parameter, and the result is rounded
to the nearest float32 by comparing exact decimal distances to the neighbouring float32 values
(ties cannot occur at this precision for these inputs).

    python tests/golden/make_decision_thresholds.py
"""
import os
import struct
from decimal import Decimal, getcontext

getcontext().prec = 60


def f32(x: float) -> float:
    return struct.unpack("<f", struct.pack("<f", x))[0]


def bits(x: float) -> int:
    return struct.unpack("<I", struct.pack("<f", x))[0]


def from_bits(b: int) -> float:
    return struct.unpack("<f", struct.pack("<I", b))[0]


def nearest_f32(x: Decimal) -> float:
    guess = f32(float(x))
    b = bits(guess)
    best = None
    for cand_bits in (b - 1, b, b + 1):
        cand = from_bits(cand_bits)
        dist = abs(Decimal(cand) - x)
        if best is None or dist < best[0]:
            best = (dist, cand)
    return best[1]


def main():
    rows = []
    for tau in (0.99, 0.9, 0.999):
        t = f32(tau)
        rows.append(("ln_tau", t, nearest_f32(Decimal(t).ln())))
    for eps in (0.2, 0.28, 0.1):
        e = f32(eps)
        rows.append(("ln_1p_eps", e, nearest_f32((Decimal(1) + Decimal(e)).ln())))
        rows.append(("ln_1m_eps", e, nearest_f32((Decimal(1) - Decimal(e)).ln())))
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "decision_thresholds.txt")
    with open(out, "w") as f:
        f.write("# float32 thresholds of the decision stage (Eq. 9: logp >= ln tau; Eq. 7 / Eq. 10 clip bounds\n"
                "# ln(1 + eps_high), ln(1 - eps_low)), correctly rounded from a 60-digit decimal logarithm of the\n"
                "# exact float32 parameter.  Written by make_decision_thresholds.py; no oracle or CUDA value.\n"
                "# kind        parameter(float32 bits)  parameter        threshold(float32 bits)  threshold\n")
        for kind, p, v in rows:
            f.write(f"{kind:<12} 0x{bits(p):08x}               {p!r:<16} 0x{bits(v):08x}               {v!r}\n")
    print(open(out).read())


if __name__ == "__main__":
    main()
