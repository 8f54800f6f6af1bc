"""Print the 24 constants floor(2^63 * 2^(-2^-i)), i = 1..24, used by the oracle's
integer 2^(-z) (Boltzmann weights of the resampling step).  80-digit decimal arithmetic
leaves more than 40 guard digits beyond the 19 digits of a 63-bit integer."""
from decimal import Decimal, getcontext, ROUND_FLOOR


def exp2_steps():
    getcontext().prec = 80
    out = []
    for i in range(1, 25):
        v = (Decimal(2) ** (-(Decimal(1) / Decimal(2 ** i)))) * Decimal(2 ** 63)
        out.append(int(v.to_integral_value(rounding=ROUND_FLOOR)))
    return out


if __name__ == "__main__":
    vals = exp2_steps()
    for r in range(0, 24, 4):
        print("    " + " ".join("0x%016Xull," % x for x in vals[r:r + 4]))
